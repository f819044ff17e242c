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


def run_fp8_chunk_case(batch, device, ks=KS, vs=VS, scratch_slack=0):
    """Quantise the existing cache with the oracle, append the chunks through the quantising append, then run
    observation-chunk attention over the fp8 pools on the GPU and in the oracle."""
    spec = batch.spec
    P = spec.page_size
    ids = batch.chunk_ids
    rows, q_indptr = batch.chunk_rows()
    k8 = oracle.fp8_quantize_rows(W.bf16_to_u16(batch.k_pool), ks)
    v8 = oracle.fp8_quantize_rows(W.bf16_to_u16(batch.v_pool), vs)
    live = np.zeros(k8.shape[:1] + k8.shape[2:3], bool)
    for t in range(spec.num_traj):
        L = int(batch.seq_lens_before[t])
        for lp in range((L + P - 1) // P):
            live[batch.page_table[t, lp], : min(P, L - lp * P)] = True
    dead = ~live                                                             # NaN codes wherever no token lives
    k8[np.broadcast_to(dead[:, None, :, None], k8.shape)] = 0x7F
    v8[np.broadcast_to(dead[:, None, :, None], v8.shape)] = 0xFF
    dk, dv = torch.from_numpy(k8.copy()).to(device), torch.from_numpy(v8.copy()).to(device)
    table, lens0 = dev_i32(batch.page_table, device), dev_i32(batch.seq_lens_before, device)
    lens1 = torch.empty_like(lens0)
    msl = int(batch.seq_lens_after.max())
    ctx = make_ctx(spec, max(1, len(ids)), msl)
    ctx.kv_append_fp8(dk, dv, table, lens0, dev_i32(batch.new_indptr, device), batch.k_new.to(device), batch.v_new.to(device),
                      ks, vs, seq_lens_out=lens1)
    after = oracle.kv_append_fp8(k8, v8, batch.page_table, batch.seq_lens_before, batch.new_indptr,
                                 W.bf16_to_u16(batch.k_new), W.bf16_to_u16(batch.v_new), ks, vs)
    q = batch.q_new[torch.from_numpy(rows)].contiguous()
    out = torch.full_like(q, float("nan"), device=device)
    lse = torch.full((q.shape[0], spec.num_q_heads), float("nan"), device=device)
    need = rollart.obs_chunk_fp8_scratch_size(len(ids), spec.num_kv_heads, P, msl)
    scratch = torch.full((need + scratch_slack,), 0xFF, dtype=torch.uint8, device=device)      # bf16 NaN everywhere
    ctx.obs_chunk_attn_fp8(dk, dv, table, lens1, dev_i32(q_indptr, device), q.to(device), spec.sm_scale, ks, vs, msl, out,
                           scratch, lse=lse, traj_ids=dev_i32(ids, device))
    ctx.check()
    assert np.array_equal(dk.cpu().numpy(), k8) and np.array_equal(dv.cpu().numpy(), v8), "the call must not touch the pools"
    ref_o, ref_l = oracle.obs_chunk_attn_fp8(k8, v8, batch.page_table, after, q_indptr, W.bf16_to_u16(q), spec.sm_scale, ks, vs,
                                             traj_ids=ids)
    assert_attn_close(out, ref_o, spec.name + " fp8 chunk")
    assert_lse_close(lse, ref_l, spec.name + " fp8 chunk")
    return ctx, (dk, dv, table, lens1), (q, q_indptr, ids, msl), out


def test_fp8_chunk_shrunk_mixed_batch(cuda_device):
    run_fp8_chunk_case(W.make_batch(W.shrink(W.CONFIGS[4], 8, 16, 8), seed=41), cuda_device)[0].close()


def test_fp8_chunk_recompute_from_empty_cache(cuda_device):
    batch = W.make_batch(W.shrink(W.RECOMPUTE, 5, 16), seed=46)
    run_fp8_chunk_case(batch, cuda_device)[0].close()


@pytest.mark.parametrize("P,hq,hkv", [(16, 8, 2), (32, 7, 1), (64, 16, 1), (16, 3, 3)])
def test_fp8_chunk_edges(cuda_device, P, hq, hkv):
    prior = [0, 0, 1, P - 1, P, 5, 130, 64]
    n_new = [1, P + 3, P, 2, 1, 130, 31, 128]
    spec = dataclasses.replace(W.CONFIGS[4], page_size=P, num_traj=len(prior), num_q_heads=hq, num_kv_heads=hkv,
                               name=f"fp8_chunk_edge_{P}_{hq}_{hkv}")
    batch = W.make_layout(spec, seed=3)
    batch.seq_lens_before = np.array(prior, np.int32)
    batch.n_new = np.array(n_new, np.int32)
    batch.is_chunk[:] = True
    batch.new_indptr = np.concatenate([[0], np.cumsum(batch.n_new)]).astype(np.int32)
    pages = (batch.seq_lens_before + batch.n_new + P - 1) // P
    batch.page_table, batch.num_pages = W.build_page_table(pages.astype(np.int64), 0.3, np.random.default_rng(2))
    W.fill_tensors(batch)
    run_fp8_chunk_case(batch, cuda_device, scratch_slack=4096)[0].close()


def test_fp8_chunk_last_row_agrees_with_fp8_decode_and_errors_are_reported(cuda_device):
    batch = W.make_batch(W.shrink(W.CONFIGS[4], 6, 32, 16), seed=77)
    spec = batch.spec
    ctx, (dk, dv, table, lens1), (q, q_indptr, ids, msl), out = run_fp8_chunk_case(batch, cuda_device)
    # the last row of a chunk sees the whole context: the decode kernel must agree within a few bf16 ulps
    last = torch.from_numpy(q_indptr[1:].astype(np.int64) - 1)
    qd = q[last].contiguous().to(cuda_device)
    od = torch.empty_like(qd)
    ctx.decode_attn_fp8(dk, dv, table, lens1, qd, spec.sm_scale, KS, VS, msl, od, traj_ids=dev_i32(ids, cuda_device))
    ctx.check()
    a, b = out[last.to(cuda_device)].float(), od.float()
    assert torch.all((a - b).abs() <= 2e-2 * b.abs() + 2e-3)
    qi = dev_i32(q_indptr, cuda_device)
    tid = dev_i32(ids, cuda_device)
    need = rollart.obs_chunk_fp8_scratch_size(len(ids), spec.num_kv_heads, spec.page_size, msl)
    scratch = torch.empty(need, dtype=torch.uint8, device=cuda_device)
    qg = q.to(cuda_device)
    with pytest.raises(rollart.RollartError) as e:          # cannot hold a single page: refused on the host
        ctx.obs_chunk_attn_fp8(dk, dv, table, lens1, qi, qg, spec.sm_scale, KS, VS, msl, out, scratch[:4096], traj_ids=tid)
    assert e.value.status == rollart.ERR_WORKSPACE
    # exactly the pages the listed contexts hold: enough; one page fewer: the device reports it and skips what does not fit
    P = spec.page_size
    pages = int(((batch.seq_lens_after[ids].astype(np.int64) + P - 1) // P).sum())
    exact = rollart.obs_chunk_fp8_scratch_size(len(ids), spec.num_kv_heads, P, msl, total_pages=pages)
    assert exact < need
    out2 = torch.full_like(out, float("nan"))
    ctx.obs_chunk_attn_fp8(dk, dv, table, lens1, qi, qg, spec.sm_scale, KS, VS, msl, out2, scratch[:exact], traj_ids=tid)
    ctx.check()
    assert torch.equal(out2.view(torch.int16), out.view(torch.int16))
    short = rollart.obs_chunk_fp8_scratch_size(len(ids), spec.num_kv_heads, P, msl, total_pages=pages - 1)
    ctx.obs_chunk_attn_fp8(dk, dv, table, lens1, qi, qg, spec.sm_scale, KS, VS, msl, out2, scratch[:short], traj_ids=tid)
    assert ctx.status() == rollart.ERR_WORKSPACE and "scratch" in ctx.last_error()
    for ks, vs in [(0.0, 1.0), (1.0, float("inf")), (float("nan"), 1.0)]:
        with pytest.raises(rollart.RollartError):
            ctx.obs_chunk_attn_fp8(dk, dv, table, lens1, qi, qg, spec.sm_scale, ks, vs, msl, out, scratch, traj_ids=tid)
    # a page id out of range and a length above the bound are device-side errors, nothing is read through them
    bad_table = table.clone()
    bad_table[int(ids[0]), 0] = dk.shape[0] + 5
    ctx.obs_chunk_attn_fp8(dk, dv, bad_table, lens1, qi, qg, spec.sm_scale, KS, VS, msl, out, scratch, traj_ids=tid)
    assert ctx.status() == rollart.ERR_BOUNDS and "obs_chunk_attn" in ctx.last_error()
    ctx.obs_chunk_attn_fp8(dk, dv, table, lens1, qi, qg, spec.sm_scale, KS, VS, 64, out, scratch, traj_ids=tid)
    assert ctx.status() == rollart.ERR_BOUNDS
    ctx.close()


def test_fp8_expansion_is_exact_for_every_code(cuda_device):
    """The bf16 copy the chunk call makes of the cache, read back from the scratch buffer: every one of the 256 codes
    (NaN codes included, in live slots here) against the oracle's decoder, bit for bit."""
    P, H, D = 16, 3, 128
    rng = np.random.default_rng(5)
    lens = np.array([37, 16, 1, 80], np.int32)
    pages = (lens.astype(np.int64) + P - 1) // P
    table, num_pages = W.build_page_table(pages, 0.25, np.random.default_rng(4))
    k8 = rng.integers(0, 256, (num_pages, H, P, D)).astype(np.uint8)
    v8 = rng.integers(0, 256, (num_pages, H, P, D)).astype(np.uint8)
    k8[table[0, 0], 0, 0, :] = np.arange(128, dtype=np.uint8)                  # every code at least once
    k8[table[0, 0], 0, 1, :] = np.arange(128, 256, dtype=np.uint8)
    spec = dataclasses.replace(W.CONFIGS[0], page_size=P, num_traj=4, num_q_heads=6, num_kv_heads=H, name="fp8_expand")
    msl = int(lens.max())
    ctx = make_ctx(spec, 4, msl)
    need = rollart.obs_chunk_fp8_scratch_size(4, H, P, msl)
    scratch = torch.zeros(need, dtype=torch.uint8, device=cuda_device)
    q = torch.zeros(4, 6, D, dtype=torch.bfloat16, device=cuda_device)
    out = torch.empty_like(q)
    ctx.obs_chunk_attn_fp8(torch.from_numpy(k8).to(cuda_device), torch.from_numpy(v8).to(cuda_device), dev_i32(table, cuda_device),
                           dev_i32(lens, cuda_device), dev_i32(np.arange(5), cuda_device), q, 1.0, 1.0, 1.0, msl, out, scratch)
    ctx.check()
    # worst-case sizing: each pool holds 4 * ppi pages; the items' pages are packed in call order
    ppi = (msl + P - 1) // P
    pool_bytes = 4 * ppi * H * P * D * 2
    sc = scratch.cpu().numpy()
    off_v = (pool_bytes + 255) // 256 * 256
    first = np.concatenate([[0], np.cumsum(pages)])
    for name, codes, off in (("k", k8, 0), ("v", v8, off_v)):
        got = sc[off: off + pool_bytes].view(np.uint16).reshape(4 * ppi, H, P, D)
        for i in range(4):
            for lp in range(int(pages[i])):
                want = oracle.fp8_pool_as_bf16_bits(codes[table[i, lp]])
                g = got[first[i] + lp]
                nan_w = (want & 0x7FFF) > 0x7F80
                nan_g = (g & 0x7FFF) > 0x7F80
                assert np.array_equal(nan_w, nan_g), (name, i, lp)
                assert np.array_equal(g[~nan_w], want[~nan_w]), (name, i, lp)
    ctx.close()


def test_fp8_more_items_than_one_launch_holds(cuda_device):
    # 1300 short trajectories through the fp8 append + decode (several launches per call), and 1100 chunk items of
    # 1..5 tokens through the fp8 chunk call (the second launch starts at a scratch row other than 0)
    spec = dataclasses.replace(W.CONFIGS[0], num_traj=1300, len_lo=1, len_hi=90, name="fp8_many_items")
    run_fp8_case(W.make_batch(spec, seed=71), cuda_device)
    spec = dataclasses.replace(W.CONFIGS[0], num_traj=1100, len_lo=1, len_hi=40, chunk_fraction=1.0, chunk_lo=1, chunk_hi=5,
                               name="fp8_many_chunks")
    run_fp8_chunk_case(W.make_batch(spec, seed=72), cuda_device)[0].close()


def test_fp8_empty_items_and_empty_calls(cuda_device):
    # an item with no chunk rows among live ones, and fp8 calls with nothing to do at all
    spec = dataclasses.replace(W.CONFIGS[4], num_traj=4, name="fp8_empties")
    batch = W.make_layout(W.shrink(spec, 4, 64, 16), seed=47)
    batch.is_chunk[:] = True
    batch.n_new = np.array([5, 0, 40, 1], np.int32)
    batch.new_indptr = np.concatenate([[0], np.cumsum(batch.n_new)]).astype(np.int32)
    P = batch.spec.page_size
    pages = (batch.seq_lens_before.astype(np.int64) + batch.n_new + P - 1) // P
    batch.page_table, batch.num_pages = W.build_page_table(pages, 0.3, np.random.default_rng(1))
    W.fill_tensors(batch)
    ctx, (dk, dv, table, lens1), _, _ = run_fp8_chunk_case(batch, cuda_device)
    hq, hkv = batch.spec.num_q_heads, batch.spec.num_kv_heads
    empty_q = torch.zeros(0, hq, 128, dtype=torch.bfloat16, device=cuda_device)
    empty_kv = torch.zeros(0, hkv, 128, dtype=torch.bfloat16, device=cuda_device)
    empty_codes = torch.zeros(0, hkv, 128, dtype=torch.uint8, device=cuda_device)
    scratch = torch.empty(1 << 20, dtype=torch.uint8, device=cuda_device)
    n0 = ctx.launch_count
    ctx.obs_chunk_attn_fp8(dk, dv, table, lens1, dev_i32([0], cuda_device), empty_q, 0.1, KS, VS, 100, empty_q.clone(), scratch)
    ctx.decode_attn_fp8(dk, dv, table, lens1, empty_q, 0.1, KS, VS, 100, empty_q.clone(), traj_ids=dev_i32([], cuda_device))
    ctx.append_decode_attn_fp8(dk, dv, table, lens1, empty_kv, empty_kv.clone(), empty_q, 0.1, KS, VS, 100, empty_q.clone(),
                               traj_ids=dev_i32([], cuda_device))
    ctx.kv_append_fp8(dk, dv, table, lens1, dev_i32([0], cuda_device), empty_kv, empty_kv.clone(), KS, VS)
    ctx.kv_append_fp8_codes(dk, dv, table, lens1, dev_i32([0], cuda_device), empty_codes, empty_codes.clone())
    ctx.kv_gather_fp8(dk, dv, table, lens1, dev_i32([0], cuda_device), empty_codes, empty_codes.clone())
    ctx.check()
    assert ctx.launch_count == n0          # nothing was enqueued
    ctx.close()


def test_fp8_reruns_are_bit_identical(cuda_device):
    # fixed schedule, fixed merge and combine order, no float atomics: the fp8 decode and chunk calls repeat bit for bit
    batch = W.make_batch(W.shrink(W.CONFIGS[4], 10, 8, 16), seed=88)
    spec = batch.spec
    ctx, (dk, dv, table, lens1), (q, q_indptr, ids, msl), out = run_fp8_chunk_case(batch, cuda_device)
    need = rollart.obs_chunk_fp8_scratch_size(len(ids), spec.num_kv_heads, spec.page_size, msl)
    scratch = torch.empty(need, dtype=torch.uint8, device=cuda_device)
    qg, qi, tid = q.to(cuda_device), dev_i32(q_indptr, cuda_device), dev_i32(ids, cuda_device)
    lse0 = torch.empty(q.shape[0], spec.num_q_heads, device=cuda_device)
    for _ in range(3):
        o = torch.full_like(out, float("nan"))
        lse = torch.full_like(lse0, float("nan"))
        ctx.obs_chunk_attn_fp8(dk, dv, table, lens1, qi, qg, spec.sm_scale, KS, VS, msl, o, scratch, lse=lse, traj_ids=tid)
        ctx.check()
        assert torch.equal(o.view(torch.int16), out.view(torch.int16))
        lse0 = lse if _ == 0 else lse0
        assert torch.equal(lse, lse0)
    dids = dev_i32(batch.decode_ids, cuda_device)
    qd = batch.q_new[torch.from_numpy(batch.decode_rows())].contiguous().to(cuda_device)
    first = None
    for _ in range(3):
        o = torch.full_like(qd, float("nan"))
        ctx.decode_attn_fp8(dk, dv, table, lens1, qd, spec.sm_scale, KS, VS, msl, o, traj_ids=dids)
        ctx.check()
        first = o if first is None else first
        assert torch.equal(o.view(torch.int16), first.view(torch.int16))
    ctx.close()
