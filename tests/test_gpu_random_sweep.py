"""Seeded random sweep of small shapes through every attention call, against the oracle.

The enumerated edge lists of the other files fix one dimension at a time; here page size, head counts, group size,
lengths (with zeros, ones and page edges mixed in), the decode / chunk split and the chunk lengths are all drawn
together, one mixed batch per seed, and the same batch goes through the bf16 and the fp8 calls."""
import dataclasses

import numpy as np
import pytest

from paper_2512_22560_b200 import workloads as W
from test_gpu_chunk import run_chunk_case
from test_gpu_decode import run_decode_case
from test_gpu_fp8 import run_fp8_case, run_fp8_chunk_case

pytestmark = pytest.mark.gpu


def random_batch(seed: int) -> W.Batch:
    rng = np.random.default_rng(1000 + seed)
    P = int(rng.choice([16, 32, 64]))
    hkv = int(rng.integers(1, 5))
    g = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 16]))
    T = int(rng.integers(2, 13))
    special = np.array([0, 1, 2, P - 1, P, P + 1, 63, 64, 65, 127, 128, 129, 4 * P, 4 * P + 1])
    lens = np.where(rng.random(T) < 0.5, rng.choice(special, T), rng.integers(0, 900, T)).astype(np.int32)
    is_chunk = rng.random(T) < 0.5
    is_chunk[0], is_chunk[1] = True, False                       # at least one of each kind
    n_special = np.array([1, 2, P - 1, P, P + 1, 31, 32, 33, 64, 127, 128, 129])
    n_chunk = np.where(rng.random(T) < 0.5, rng.choice(n_special, T), rng.integers(1, 300, T))
    n_new = np.where(is_chunk, n_chunk, 1).astype(np.int32)
    spec = dataclasses.replace(W.CONFIGS[0], page_size=P, num_traj=T, num_q_heads=g * hkv, num_kv_heads=hkv,
                               name=f"sweep{seed}_p{P}_h{hkv}_g{g}_t{T}")
    batch = W.make_layout(spec, seed=seed)
    batch.seq_lens_before, batch.n_new, batch.is_chunk = lens, n_new, is_chunk
    batch.new_indptr = np.concatenate([[0], np.cumsum(n_new)]).astype(np.int32)
    pages = (lens.astype(np.int64) + n_new + P - 1) // P
    batch.page_table, batch.num_pages = W.build_page_table(pages, 0.3, np.random.default_rng(seed))
    return W.fill_tensors(batch)


@pytest.mark.parametrize("seed", range(16))
def test_random_mixed_batch_bf16(cuda_device, seed):
    batch = random_batch(seed)
    run_decode_case(batch, cuda_device)
    _, ctx, _, _ = run_chunk_case(random_batch(seed), cuda_device)
    ctx.close()


@pytest.mark.parametrize("seed", range(16))
def test_random_mixed_batch_fp8(cuda_device, seed):
    run_fp8_case(random_batch(seed), cuda_device)
    run_fp8_chunk_case(random_batch(seed), cuda_device)[0].close()


@pytest.mark.parametrize("seed", range(10))
def test_random_groups(cuda_device, seed):
    # the group calls (bf16 and fp8) on random shapes, group sizes and shared fractions
    from test_gpu_group_decode import run_fp8_group_case, run_group_case
    rng = np.random.default_rng(2000 + seed)
    P = int(rng.choice([16, 32, 64]))
    hkv = int(rng.integers(1, 5))
    g = int(rng.choice([1, 2, 4, 7, 8, 16]))
    T = int(rng.integers(2, 40))
    lo = int(rng.integers(1, 200))
    spec = dataclasses.replace(W.CONFIGS[0], page_size=P, num_traj=T, num_q_heads=g * hkv, num_kv_heads=hkv,
                               len_lo=lo, len_hi=lo + int(rng.integers(1, 800)), name=f"gsweep{seed}_p{P}_h{hkv}_g{g}_t{T}")
    group_size = int(rng.choice([1, 2, 3, 8, 20]))
    fraction = float(rng.choice([0.0, 0.3, 0.75, 1.0]))
    run_group_case(spec, 50 + seed, group_size, fraction, cuda_device)
    run_fp8_group_case(spec, 50 + seed, group_size, fraction, cuda_device)


@pytest.mark.parametrize("seed", range(12))
def test_random_chunks_with_wild_scores(cuda_device, seed):
    # The chunk half of a random batch with keys whose magnitudes are all over the place: a heavy-tailed gain per key,
    # runs of 64 loud or quiet keys, and a few keys that score the same enormous value for every row (a constant
    # component in the queries).  The moving reference max, its rescaling of the accumulator and the checks that guard
    # both kinds of exponential all get exercised; the results are close to one-hot, so a wrong key would show.
    import torch
    batch = random_batch(100 + seed)
    rng = np.random.default_rng(3000 + seed)
    P = batch.spec.page_size
    batch.q_new[:, :, 0] = 3.0
    for t in range(batch.spec.num_traj):
        L = int(batch.seq_lens_before[t])
        if L == 0:
            continue
        gain = np.exp(rng.normal(0.0, 1.5, L))
        for b0 in range(0, L, 64):
            r = rng.random()
            if r < 0.15:
                gain[b0:b0 + 64] *= 30.0
            elif r < 0.3:
                gain[b0:b0 + 64] *= 0.01
        lone = rng.choice(L, size=min(L, int(rng.integers(0, 4))), replace=False)
        for pos in range(L):
            pg = int(batch.page_table[t, pos // P])
            if pos in lone:
                key = torch.zeros(128)
                key[0] = float(rng.choice([60.0, 150.0, 300.0, 900.0])) / (3.0 * batch.spec.sm_scale * 1.4426950408889634)
                batch.k_pool[pg, :, pos % P, :] = key.to(torch.bfloat16)
            else:
                batch.k_pool[pg, :, pos % P, :] = (batch.k_pool[pg, :, pos % P, :].float() * float(min(gain[pos], 200.0))).to(torch.bfloat16)
    _, ctx, _, _ = run_chunk_case(batch, cuda_device)
    ctx.close()
