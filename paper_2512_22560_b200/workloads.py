"""Seeded synthetic rollout batches: trajectory lengths, page tables, pools, Q and new K/V.

This module only draws random inputs and lays them out; it holds none of the
attention or append arithmetic.  Both the CUDA path's tests/bench and the CPU
oracle's tests take their inputs from here.

The five workload recipes stand in for the multi-turn agentic rollouts the
paper characterises: contexts that grow by (observation, action) pairs every
turn (Sec. 6.1, EnvManager), a bimodal few-turn / many-turn mix (Sec. 3.1),
contexts up to 32k tokens in the evaluation (Sec. 7.1) and heavy-tailed
response lengths in production (Sec. 8).  No item of any public benchmark is
reproduced: only shapes and length distributions.

Layout conventions (shared by every consumer):
  pools       bf16 [num_pages][num_kv_heads][page_size][head_dim], K and V separate
  page_table  int32 [num_traj][max_pages], entry i of row t = physical page of
              logical page i; entries past the pages a trajectory owns are -1
  seq_lens    int32 [num_traj], tokens
  new rows    bf16 [total_new][heads][head_dim], trajectory t owning rows
              new_indptr[t] .. new_indptr[t+1]
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass, field
from typing import Optional, Sequence

import numpy as np
import torch

HEAD_DIM = 128
MASTER_SEED = 20251222


@dataclass(frozen=True)
class WorkloadSpec:
    """One recipe. `length_kind` selects the context-length distribution."""
    name: str
    num_traj: int
    num_q_heads: int
    num_kv_heads: int
    page_size: int
    length_kind: str              # "uniform" | "turns" | "lognormal"
    len_lo: int = 1
    len_hi: int = 1
    len_cap: int = 1 << 30
    lognormal_median: float = 8192.0
    lognormal_sigma: float = 0.8
    chunk_fraction: float = 0.0   # fraction of trajectories that receive an observation chunk
    chunk_lo: int = 64
    chunk_hi: int = 2048
    recompute: bool = False       # every trajectory re-enters with its whole context as one chunk (empty cache before)
    k_scale: float = 1.0          # multiplier on K data
    sm_scale: float = 1.0 / math.sqrt(HEAD_DIM)
    spare_pages: float = 0.125
    head_dim: int = HEAD_DIM


CONFIGS = (
    WorkloadSpec("cfg0_tiny_decode", 4, 8, 2, 16, "uniform", len_lo=64, len_hi=512),
    WorkloadSpec("cfg1_7b_gqa_decode", 64, 28, 4, 16, "turns", len_cap=16384,
                 k_scale=1.0 / math.sqrt(HEAD_DIM), sm_scale=1.0),
    WorkloadSpec("cfg2_32b_gqa_decode", 256, 64, 8, 16, "lognormal", len_lo=1, len_cap=32768,
                 lognormal_median=8192.0, lognormal_sigma=0.8),
    WorkloadSpec("cfg3_long_horizon_decode", 32, 64, 4, 64, "uniform", len_lo=32768, len_hi=131072),
    WorkloadSpec("cfg4_mixed_multiturn", 128, 32, 8, 16, "uniform", len_lo=1024, len_hi=24576,
                 chunk_fraction=0.5, chunk_lo=64, chunk_hi=2048),
)


# KV-cache recomputation after a weight update (Sec. 6.2, step "recomp" of the asynchronous training
# protocol): every in-flight trajectory rebuilds its cache, i.e. a causal prefill of its whole context
# onto empty pages.  Same calls as the observation chunk, with no prior context.
RECOMPUTE = WorkloadSpec("recompute_inflight", 16, 32, 8, 16, "uniform", len_lo=4096, len_hi=32768, recompute=True)


# Decode step of GRPO groups under prefix caching (Sec. 7.1: group size 8, prefix caching on the rollout
# engine): 64 groups of 8 trajectories with the 7B-like head shape; share_group_prefix() makes the
# members of a group alias the pages of a common prompt prefix.
GROUP_DECODE = WorkloadSpec("grpo_group8_decode", 512, 28, 4, 16, "turns", len_cap=16384,
                            k_scale=1.0 / math.sqrt(HEAD_DIM), sm_scale=1.0)
GROUP_SIZE = 8
GROUP_SHARED_FRACTION = 0.5       # of the shortest member's context


def shrink(spec: WorkloadSpec, num_traj: int, len_div: int, chunk_div: int = 1) -> WorkloadSpec:
    """A smaller workload of the same shape (same heads, page size, distribution family)."""
    return dataclasses.replace(
        spec,
        name=f"{spec.name}_div{len_div}_t{num_traj}",
        num_traj=num_traj,
        len_lo=max(1, spec.len_lo // len_div),
        len_hi=max(1, spec.len_hi // len_div),
        len_cap=max(1, spec.len_cap // len_div) if spec.len_cap < (1 << 30) else spec.len_cap,
        lognormal_median=max(2.0, spec.lognormal_median / len_div),
        chunk_lo=max(1, spec.chunk_lo // chunk_div),
        chunk_hi=max(1, spec.chunk_hi // chunk_div),
    )


@dataclass
class Batch:
    spec: WorkloadSpec
    seed: int
    seq_lens_before: np.ndarray       # int32 [T]
    n_new: np.ndarray                 # int32 [T]
    is_chunk: np.ndarray              # bool  [T]
    new_indptr: np.ndarray            # int32 [T+1]
    page_table: np.ndarray            # int32 [T][max_pages]
    num_pages: int
    turns: Optional[list] = None      # per-trajectory turn boundaries (metadata only)
    # tensors (torch, on `device`)
    k_pool: Optional[torch.Tensor] = None
    v_pool: Optional[torch.Tensor] = None
    q_new: Optional[torch.Tensor] = None   # [total_new][Hq][D]
    k_new: Optional[torch.Tensor] = None   # [total_new][Hkv][D]
    v_new: Optional[torch.Tensor] = None
    needles: list = field(default_factory=list)

    @property
    def seq_lens_after(self) -> np.ndarray:
        return (self.seq_lens_before + self.n_new).astype(np.int32)

    @property
    def max_pages(self) -> int:
        return int(self.page_table.shape[1])

    @property
    def decode_ids(self) -> np.ndarray:
        return np.nonzero(~self.is_chunk)[0].astype(np.int32)

    @property
    def chunk_ids(self) -> np.ndarray:
        return np.nonzero(self.is_chunk)[0].astype(np.int32)

    def decode_rows(self, ids: Optional[Sequence[int]] = None) -> np.ndarray:
        """Row of q_new/k_new holding the single new token of each decode trajectory."""
        ids = self.decode_ids if ids is None else np.asarray(ids, dtype=np.int64)
        return self.new_indptr[ids].astype(np.int64)

    def chunk_rows(self, ids: Optional[Sequence[int]] = None):
        """(row indices into q_new, q_indptr) for the chunk trajectories `ids`, concatenated."""
        ids = self.chunk_ids if ids is None else np.asarray(ids, dtype=np.int64)
        rows = [np.arange(self.new_indptr[t], self.new_indptr[t + 1], dtype=np.int64) for t in ids]
        indptr = np.zeros(len(ids) + 1, dtype=np.int32)
        if len(ids):
            indptr[1:] = np.cumsum([len(r) for r in rows])
        flat = np.concatenate(rows) if rows else np.zeros(0, dtype=np.int64)
        return flat, indptr


def _sub_seed(seed: int, spec: WorkloadSpec, stream: int) -> int:
    # independent, reproducible sub-streams per (master seed, recipe, purpose)
    ss = np.random.SeedSequence([seed, sum(map(ord, spec.name)) & 0x7FFFFFFF, stream])
    return int(ss.generate_state(1, dtype=np.uint64)[0] & 0x7FFFFFFFFFFFFFFF)


def draw_lengths(spec: WorkloadSpec, rng: np.random.Generator):
    """Context lengths before the step, and per-trajectory turn boundaries where the recipe has turns."""
    T = spec.num_traj
    turns = None
    if spec.length_kind == "uniform":
        lens = rng.integers(spec.len_lo, spec.len_hi + 1, size=T)
    elif spec.length_kind == "lognormal":
        lens = np.rint(np.exp(rng.normal(math.log(spec.lognormal_median), spec.lognormal_sigma, size=T)))
        lens = np.clip(lens, max(1, spec.len_lo), spec.len_cap)
    elif spec.length_kind == "turns":
        lens = np.zeros(T, dtype=np.int64)
        turns = []
        for t in range(T):
            n_turns = int(rng.integers(2, 11))
            obs = rng.integers(200, 1001, size=n_turns)
            act = rng.integers(100, 501, size=n_turns)
            bounds = np.cumsum(np.stack([obs, act], axis=1).reshape(-1))
            lens[t] = min(int(bounds[-1]), spec.len_cap)
            turns.append(np.minimum(bounds, spec.len_cap).astype(np.int32))
    else:
        raise ValueError(spec.length_kind)
    return lens.astype(np.int32), turns


def build_page_table(pages_per_traj: np.ndarray, spare: float, rng: np.random.Generator):
    """Physical page ids: a seeded permutation of the pool, dealt round-robin over trajectories
    (logical page 0 of every trajectory, then logical page 1, ...), unused entries -1."""
    T = len(pages_per_traj)
    total = int(pages_per_traj.sum())
    num_pages = max(1, int(math.ceil(total * (1.0 + spare))))
    perm = rng.permutation(num_pages)[:total].astype(np.int32)
    max_pages = max(1, int(pages_per_traj.max()) if T else 1)
    table = np.full((T, max_pages), -1, dtype=np.int32)
    logical = np.arange(max_pages)[None, :].repeat(T, axis=0)
    owned = logical < pages_per_traj[:, None]
    # order of dealing: by logical page index first, then by trajectory
    order = np.argsort(logical[owned], kind="stable")
    tt, ll = np.nonzero(owned)
    table[tt[order], ll[order]] = perm
    return table, num_pages


def make_layout(spec: WorkloadSpec, seed: int = MASTER_SEED) -> Batch:
    """Lengths, chunk assignment and page table only (no tensors)."""
    rng = np.random.default_rng(_sub_seed(seed, spec, 0))
    lens, turns = draw_lengths(spec, rng)
    T = spec.num_traj
    n_new = np.ones(T, dtype=np.int32)
    is_chunk = np.zeros(T, dtype=bool)
    n_chunk = int(round(T * spec.chunk_fraction))
    if n_chunk:
        ids = rng.permutation(T)[:n_chunk]
        is_chunk[ids] = True
        n_new[ids] = rng.integers(spec.chunk_lo, spec.chunk_hi + 1, size=n_chunk)
    if spec.recompute:
        n_new = lens.copy()
        lens = np.zeros(T, dtype=np.int32)
        is_chunk[:] = True
    new_indptr = np.zeros(T + 1, dtype=np.int32)
    new_indptr[1:] = np.cumsum(n_new)
    pages = (lens.astype(np.int64) + n_new + spec.page_size - 1) // spec.page_size
    table, num_pages = build_page_table(pages, spec.spare_pages, rng)
    return Batch(spec, seed, lens, n_new, is_chunk, new_indptr, table, num_pages, turns)


def _randn_bf16(shape, gen: torch.Generator, device, scale: float = 1.0) -> torch.Tensor:
    numel = int(np.prod(shape))
    out = torch.empty(numel, dtype=torch.bfloat16, device=device)
    step = 1 << 28  # bound the fp32 temporary
    for s in range(0, numel, step):
        e = min(numel, s + step)
        x = torch.randn(e - s, dtype=torch.float32, device=device, generator=gen)
        if scale != 1.0:
            x *= scale
        out[s:e] = x.to(torch.bfloat16)
    return out.view(*shape)


def fill_tensors(batch: Batch, device="cpu") -> Batch:
    """Pools ~ N(0,1) everywhere (so the context before the step is N(0,1) and every
    unowned slot holds arbitrary finite values), Q / new K / new V ~ N(0,1); K times k_scale."""
    spec = batch.spec
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(_sub_seed(batch.seed, spec, 1))
    shape = (batch.num_pages, spec.num_kv_heads, spec.page_size, spec.head_dim)
    batch.k_pool = _randn_bf16(shape, gen, dev, spec.k_scale)
    batch.v_pool = _randn_bf16(shape, gen, dev)
    total_new = int(batch.new_indptr[-1])
    batch.q_new = _randn_bf16((total_new, spec.num_q_heads, spec.head_dim), gen, dev)
    batch.k_new = _randn_bf16((total_new, spec.num_kv_heads, spec.head_dim), gen, dev, spec.k_scale)
    batch.v_new = _randn_bf16((total_new, spec.num_kv_heads, spec.head_dim), gen, dev)
    return batch


def make_batch(spec: WorkloadSpec, seed: int = MASTER_SEED, device="cpu") -> Batch:
    return fill_tensors(make_layout(spec, seed), device)


# ---------------------------------------------------------------------------------------------
# Test-only shaping of inputs (still no method arithmetic: bit patterns and copies).
# ---------------------------------------------------------------------------------------------
POISON_PATTERNS = (0x7FC0, 0x7F80, 0xFF80, 0x7F7F, 0xFFC1)  # NaN, +Inf, -Inf, 3.39e38, -NaN


def slot_owner_mask(batch: Batch, lens: np.ndarray) -> torch.Tensor:
    """bool [num_pages][page_size]: True where a slot holds one of the first lens[t] tokens of some trajectory."""
    P = batch.spec.page_size
    live = torch.zeros(batch.num_pages, P, dtype=torch.bool)
    for t in range(len(lens)):
        L = int(lens[t])
        if L <= 0:
            continue
        npg = (L + P - 1) // P
        ids = torch.from_numpy(batch.page_table[t, :npg].astype(np.int64))
        live[ids] = True
        tail = L - (npg - 1) * P
        live[ids[-1], tail:] = False
    return live


def poison_dead_slots(batch: Batch, lens: np.ndarray) -> None:
    """Overwrite every slot that is not among the first lens[t] tokens of its owner (page tails,
    unowned pages) with NaN / Inf / huge bit patterns, cycling through POISON_PATTERNS."""
    live = slot_owner_mask(batch, lens).to(batch.k_pool.device)
    dead = ~live                                            # [pages][P]
    pat = torch.tensor(POISON_PATTERNS, dtype=torch.int32)
    idx = (torch.arange(batch.num_pages)[:, None] * 3 + torch.arange(batch.spec.page_size)[None, :]) % len(pat)
    bits = pat[idx].to(torch.int16).to(batch.k_pool.device)  # [pages][P]
    for pool in (batch.k_pool, batch.v_pool):
        raw = pool.view(torch.int16)                         # [pages][H][P][D]
        m = dead[:, None, :, None].expand_as(raw)
        raw[m] = bits[:, None, :, None].expand_as(raw)[m]


def plant_needles(batch: Batch, positions_per_traj: dict, beta: float = 3.0) -> None:
    """Make chosen context positions dominate the softmax of the decode query (outputs become O(1)):
    K at (t, pos, kv head h) := beta * q of the (pos mod g)-th q head of h's group, for the
    trajectory's last new token; V there is left as drawn.  Must be called before the append, on
    positions < seq_lens_before[t], or on the new rows themselves via k_new (pos == -1)."""
    spec = batch.spec
    g = spec.num_q_heads // spec.num_kv_heads
    P = spec.page_size
    for t, positions in positions_per_traj.items():
        qrow = int(batch.new_indptr[t + 1]) - 1
        q = batch.q_new[qrow].float().view(spec.num_kv_heads, g, spec.head_dim)
        for pos in positions:
            pos = int(pos)
            kvec = (beta * q[:, pos % g, :]).to(torch.bfloat16)      # [Hkv][D]
            if pos < int(batch.seq_lens_before[t]):
                pg = int(batch.page_table[t, pos // P])
                batch.k_pool[pg, :, pos % P, :] = kvec
            else:
                row = int(batch.new_indptr[t]) + (pos - int(batch.seq_lens_before[t]))
                batch.k_new[row] = kvec
            batch.needles.append((t, pos))


def share_group_prefix(batch: Batch, group_size: int, fraction: float):
    """Turns consecutive runs of `group_size` trajectories into groups that share a prompt prefix, the
    way prefix caching leaves the members of a GRPO group (paper Sec. 7.1: group size 8, prefix caching
    on): the members' page-table rows are made to list the first member's pages for the first
    floor(fraction * shortest member length / page_size) pages.  Returns (group_indptr, shared_lens),
    both int32; shared_lens is in tokens.  Only indices are rewritten: pool contents stay as they are,
    the pages the other members owned there are simply no longer referenced."""
    T, P = batch.spec.num_traj, batch.spec.page_size
    starts = list(range(0, T, group_size)) + [T]
    indptr = np.asarray(starts, dtype=np.int32)
    shared = np.zeros(len(starts) - 1, dtype=np.int32)
    for gi in range(len(starts) - 1):
        a, b = starts[gi], starts[gi + 1]
        pages = int(int(batch.seq_lens_before[a:b].min()) * fraction) // P
        batch.page_table[a + 1:b, :pages] = batch.page_table[a, :pages]
        shared[gi] = pages * P
    return indptr, shared


def extract_trajs(batch: Batch, ids: Sequence[int]) -> Batch:
    """Host-side sub-batch holding only trajectories `ids`, with their pages renumbered 0..n-1
    (in a compact pool, CPU tensors).  Used to hand a sample of a large device-resident batch
    to a CPU checker."""
    ids = np.asarray(ids, dtype=np.int64)
    spec = dataclasses.replace(batch.spec, num_traj=len(ids), name=batch.spec.name + "_sample")
    P = spec.page_size
    pages = (batch.seq_lens_before[ids].astype(np.int64) + batch.n_new[ids] + P - 1) // P
    phys = np.concatenate([batch.page_table[t, :n] for t, n in zip(ids, pages)]).astype(np.int64)
    table = np.full((len(ids), max(1, int(pages.max()))), -1, dtype=np.int32)
    o = 0
    for i, n in enumerate(pages):
        table[i, :n] = np.arange(o, o + n, dtype=np.int32)
        o += int(n)
    new_indptr = np.zeros(len(ids) + 1, dtype=np.int32)
    new_indptr[1:] = np.cumsum(batch.n_new[ids])
    rows = np.concatenate([np.arange(batch.new_indptr[t], batch.new_indptr[t + 1]) for t in ids]).astype(np.int64)
    sub = Batch(spec, batch.seed, batch.seq_lens_before[ids].copy(), batch.n_new[ids].copy(),
                batch.is_chunk[ids].copy(), new_indptr, table, int(len(phys)))
    pidx = torch.from_numpy(phys).to(batch.k_pool.device)
    ridx = torch.from_numpy(rows).to(batch.k_pool.device)
    sub.k_pool = batch.k_pool.index_select(0, pidx).cpu()
    sub.v_pool = batch.v_pool.index_select(0, pidx).cpu()
    sub.q_new = batch.q_new.index_select(0, ridx).cpu()
    sub.k_new = batch.k_new.index_select(0, ridx).cpu()
    sub.v_new = batch.v_new.index_select(0, ridx).cpu()
    return sub


def bf16_to_u16(t: torch.Tensor) -> np.ndarray:
    """Bit view of a bf16 tensor as a contiguous uint16 numpy array (host)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def u16_to_bf16(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
