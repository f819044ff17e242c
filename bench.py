#!/usr/bin/env python
"""Benchmark of the rollout-attention hot path on B200.

A step is one pass of the engine step's attention part over one synthetic batch of
trajectories: KV append of one new token per trajectory, then decode attention over each
trajectory's whole paged context (split over thread blocks, merged by the log-sum-exp combine).
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2512_22560_b200 import workloads as W  # noqa: E402

METRIC = "paged-KV decode attention: achieved HBM GB/s (% of B200 peak), decode tokens/s"
UNIT = "decode tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            with open(path) as f:
                return float(json.load(f)["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def measured_traffic(workload: str, seed: int):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the tracked record of an
    ncu capture.  The record names the workload, the seed and the SHA-256 of the kernel's source files at capture time:
    any other workload or seed, or a source file that has changed since, gives None (the counters no longer describe
    the kernel that runs)."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "decode_splitkv_traffic.json")
    try:
        with open(path) as f:
            rec = json.load(f)
        if rec["workload"] != workload or int(rec["seed"]) != int(seed):
            return None
        for rel, digest in rec["source_sha256"].items():
            with open(os.path.join(ROOT, rel), "rb") as f:
                if hashlib.sha256(f.read()).hexdigest() != digest:
                    return None
        return float(rec["dram_bytes_per_launch"])
    except Exception:
        return None


def decode_algorithmic_bytes(spec: W.WorkloadSpec, lens_after: np.ndarray) -> int:
    """K and V of every context token read once per kv head (shared by the group's q heads),
    Q in and O out, and the page-table entries that are needed."""
    kv = int(lens_after.astype(np.int64).sum()) * 2 * spec.num_kv_heads * spec.head_dim * 2
    qo = 2 * len(lens_after) * spec.num_q_heads * spec.head_dim * 2
    pt = 4 * int(((lens_after.astype(np.int64) + spec.page_size - 1) // spec.page_size).sum())
    return kv + qo + pt


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs (read only)."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.source = "nvidia-smi"
        self._stop = threading.Event()
        self._t = threading.Thread(target=self._run, daemon=True)

    def _nvml_handle(self):
        """NVML handle of torch's device `index` (by UUID, so a CUDA_VISIBLE_DEVICES remapping does not matter)."""
        import pynvml
        pynvml.nvmlInit()
        try:
            uuid = str(torch.cuda.get_device_properties(self.index).uuid)
            return pynvml, pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
        except Exception:
            return pynvml, pynvml.nvmlDeviceGetHandleByIndex(self.index)

    def _run(self):
        # NVML queries (read only) take well under a millisecond, so a 0.2 s timed region still gets some twenty
        # samples; nvidia-smi, at ~0.1 s per call, is the fallback
        try:
            nv, h = self._nvml_handle()
            bits = (nv.nvmlClocksThrottleReasonHwSlowdown, nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                    nv.nvmlClocksThrottleReasonSwThermalSlowdown, nv.nvmlClocksThrottleReasonSwPowerCap)
            mx = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            self.source = "nvml"
            while not self._stop.is_set():
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                self.rows.append([str(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)), str(mx),
                                  "%.1f" % (nv.nvmlDeviceGetPowerUsage(h) / 1000.0)] +
                                 ["Active" if r & b else "Not Active" for b in bits])
                self._stop.wait(0.01)
            return
        except Exception:
            self.source = "nvidia-smi"
        while not self._stop.is_set():
            try:
                r = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                    "-i", str(self.index)], capture_output=True, text=True, timeout=5)
                if r.returncode == 0 and r.stdout.strip():
                    self.rows.append([x.strip() for x in r.stdout.strip().split(",")])
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._t.join(timeout=6)

    def summary(self):
        sm = [float(r[0]) for r in self.rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) > 3 + i and r[3 + i].lower().startswith("active") for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(self.rows), "source": self.source}


class DecodeWorkload:
    """Device-resident state of one workload plus the two calls of a step."""

    def __init__(self, spec: W.WorkloadSpec, seed: int, device: torch.device, ids=None):
        from paper_2512_22560_b200 import rollart
        self.spec = spec
        self.device = device
        b = W.make_batch(spec, seed=seed, device=device)
        self.batch = b
        ids = b.decode_ids if ids is None else ids
        self.ids = ids
        i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
        self.table = i32(b.page_table)
        self.lens0 = i32(b.seq_lens_before)
        self.lens1 = i32(b.seq_lens_after)          # overwritten by the append of the ids below
        self.traj_ids = i32(ids)
        rows = torch.from_numpy(b.decode_rows(ids)).to(device)
        self.q = b.q_new[rows].contiguous()
        self.k_new = b.k_new[rows].contiguous()
        self.v_new = b.v_new[rows].contiguous()
        self.indptr = i32(np.arange(len(ids) + 1))
        self.out = torch.empty_like(self.q)
        self.max_seq_len = int(b.seq_lens_after[ids].max())
        self.ctx = rollart.Context(device.index or 0, rollart.workspace_size(len(ids), spec.num_q_heads, spec.num_kv_heads,
                                                                            self.max_seq_len))
        self.lens_after_host = b.seq_lens_after[ids]
        self.bytes = decode_algorithmic_bytes(spec, self.lens_after_host)
        self.n_items = len(ids)

    def append(self):
        self.ctx.kv_append(self.batch.k_pool, self.batch.v_pool, self.table, self.lens0, self.indptr, self.k_new, self.v_new,
                           traj_ids=self.traj_ids, seq_lens_out=self.lens1)

    def decode(self):
        self.ctx.decode_attn(self.batch.k_pool, self.batch.v_pool, self.table, self.lens1, self.q, self.spec.sm_scale,
                             self.max_seq_len, self.out, traj_ids=self.traj_ids)

    def step(self):
        """One decode step: the fused call stores the new token's K/V and attends, in one launch."""
        self.ctx.append_decode_attn(self.batch.k_pool, self.batch.v_pool, self.table, self.lens0, self.k_new, self.v_new, self.q,
                                    self.spec.sm_scale, self.max_seq_len, self.out, traj_ids=self.traj_ids,
                                    seq_lens_out=self.lens1)

    def time_steps(self, steps: int, warmup: int, min_total_ms: float = 0.0):
        """Times loops of exactly `steps` back-to-back steps (two CUDA events per loop, nothing inside the loop).  A loop
        that lasts less than min_total_ms is repeated until the loops together last about that long, so that a short
        `steps` does not rest on one window of a few milliseconds.  Returns the list of loop times in ms.  A step is
        one kernel launch, so loop time / steps is the average launch period."""
        for _ in range(warmup):
            self.step()
        torch.cuda.synchronize(self.device)

        def loops(n):
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
            for a, b in ev:
                a.record()
                for _ in range(steps):
                    self.step()
                b.record()
            torch.cuda.synchronize(self.device)
            return [a.elapsed_time(b) for a, b in ev]

        times = loops(1)
        if times[0] < min_total_ms:
            times += loops(min(2000, int(np.ceil(min_total_ms / max(times[0], 1e-3))) - 1))
        self.ctx.check()
        return times

    def time_fp8_steps(self, steps: int, warmup: int, k_scale: float = 0.03, v_scale: float = 0.03):
        """The same step over fp8 (E4M3) pools: quantised append of the new token + fp8 decode attention in one launch.
        The pools are the bf16 pools quantised with the given scales.  Returns (ms per step, KV bytes read per step)."""
        b = self.batch
        k8 = (b.k_pool.float() * (1.0 / k_scale)).to(torch.float8_e4m3fn).view(torch.uint8)
        v8 = (b.v_pool.float() * (1.0 / v_scale)).to(torch.float8_e4m3fn).view(torch.uint8)

        def step():
            self.ctx.append_decode_attn_fp8(k8, v8, self.table, self.lens0, self.k_new, self.v_new, self.q, self.spec.sm_scale,
                                            k_scale, v_scale, self.max_seq_len, self.out, traj_ids=self.traj_ids,
                                            seq_lens_out=self.lens1)

        for _ in range(warmup):
            step()
        torch.cuda.synchronize(self.device)
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(steps):
            step()
        t1.record()
        torch.cuda.synchronize(self.device)
        self.ctx.check()
        kv_bytes = int(self.lens_after_host.astype(np.int64).sum()) * 2 * self.spec.num_kv_heads * self.spec.head_dim
        return t0.elapsed_time(t1) / steps, kv_bytes + 2 * self.q.numel() * 2

    def time_gather(self, steps: int = 5, warmup: int = 2):
        """KV hand-off: all trajectories' caches gathered into contiguous rows.  (mean ms, bytes read + written)"""
        b = self.batch
        lens = b.seq_lens_before[self.ids]
        indptr = np.concatenate([[0], np.cumsum(lens.astype(np.int64))])
        if indptr[-1] >= 2 ** 31:
            raise ValueError("too many rows for one gather call")
        d_indptr = torch.from_numpy(indptr.astype(np.int32)).to(self.device)
        k_out = torch.empty(int(indptr[-1]), self.spec.num_kv_heads, self.spec.head_dim, dtype=torch.bfloat16, device=self.device)
        v_out = torch.empty_like(k_out)
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps)]
        for s in range(warmup + steps):
            if s >= warmup:
                ev[s - warmup][0].record()
            self.ctx.kv_gather(b.k_pool, b.v_pool, self.table, self.lens0, d_indptr, k_out, v_out, traj_ids=self.traj_ids)
            if s >= warmup:
                ev[s - warmup][1].record()
        torch.cuda.synchronize(self.device)
        self.ctx.check()
        return float(np.mean([e[0].elapsed_time(e[1]) for e in ev])), 2 * 2 * k_out.numel() * 2

    def time_e2e(self, steps: int, warmup: int):
        """Steps driven from HOST buffers through rollart_append_decode_attn_host: per step the new token's q/k/v go
        host->device from pinned memory (one buffer, one copy, enqueued by the call) and the attention output goes
        device->host (the kernel stores it into a pinned host buffer, no separate copy), inside the timed region.  The
        call's arguments are marshalled once (a decode loop rewrites the buffers' contents, not their addresses)."""
        from paper_2512_22560_b200 import rollart
        nq, nk = self.q.numel(), self.k_new.numel()
        host = torch.cat([self.q.flatten(), self.k_new.flatten(), self.v_new.flatten()]).cpu().pin_memory()
        hq, hk, hv = host[:nq].view_as(self.q), host[nq:nq + nk].view_as(self.k_new), host[nq + nk:].view_as(self.v_new)
        hout = torch.empty_like(self.out, device="cpu").pin_memory()
        staging = torch.empty(rollart.host_staging_size(self.n_items, self.spec.num_q_heads, self.spec.num_kv_heads),
                              dtype=torch.uint8, device=self.device)
        step = self.ctx.bind_append_decode_attn_host(self.batch.k_pool, self.batch.v_pool, self.table, self.lens0, hk, hv, hq,
                                                     self.spec.sm_scale, self.max_seq_len, hout, staging, traj_ids=self.traj_ids,
                                                     seq_lens_out=self.lens1)

        def one():
            step()
            torch.cuda.synchronize(self.device)     # the host consumes each step's result
        for _ in range(warmup):
            one()
        # several loops of `steps` steps, the median loop: a host-side hiccup (another tenant's burst on the host cores)
        # lands in one loop and does not move the figure
        loops = []
        for _ in range(5):
            t0 = time.perf_counter()
            for _ in range(steps):
                one()
            loops.append(time.perf_counter() - t0)
        self.ctx.check()
        return float(np.median(loops)) * 1e3, host.numel() * 2, hout.numel() * 2


class GroupDecodeWorkload:
    """GRPO groups whose members alias a shared prompt prefix: one decode step is the KV append of the new
    tokens followed by the group decode call (prefix read once per group)."""

    def __init__(self, spec: W.WorkloadSpec, seed: int, device: torch.device, group_size: int, fraction: float):
        from paper_2512_22560_b200 import rollart
        self.spec = spec
        self.device = device
        layout = W.make_layout(spec, seed)
        indptr, shared = W.share_group_prefix(layout, group_size, fraction)
        b = W.fill_tensors(layout, device)
        self.batch = b
        i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
        self.table, self.lens0, self.lens1 = i32(b.page_table), i32(b.seq_lens_before), i32(b.seq_lens_after)
        self.group_indptr, self.shared = i32(indptr), i32(shared)
        self.new_indptr = i32(b.new_indptr)
        self.q = b.q_new.contiguous()
        self.out = torch.empty_like(self.q)
        self.max_seq_len = int(b.seq_lens_after.max())
        self.n_items = spec.num_traj
        self.ctx = rollart.Context(device.index or 0, rollart.group_decode_workspace_size(
            self.n_items, spec.num_q_heads, spec.num_kv_heads, self.max_seq_len))
        per_token = 2 * spec.num_kv_heads * spec.head_dim * 2
        self.bytes_per_trajectory_definition = decode_algorithmic_bytes(spec, b.seq_lens_after)
        members = np.diff(indptr).astype(np.int64)
        self.bytes_unique = self.bytes_per_trajectory_definition - int(((members - 1).clip(min=0) * shared).sum()) * per_token

    def step_group(self):
        b = self.batch
        self.ctx.kv_append(b.k_pool, b.v_pool, self.table, self.lens0, self.new_indptr, b.k_new, b.v_new, seq_lens_out=self.lens1)
        self.ctx.group_decode_attn(b.k_pool, b.v_pool, self.table, self.lens1, self.group_indptr, self.shared, self.q,
                                   self.spec.sm_scale, self.max_seq_len, self.out)

    def step_plain(self):
        b = self.batch
        self.ctx.append_decode_attn(b.k_pool, b.v_pool, self.table, self.lens0, b.k_new, b.v_new, self.q, self.spec.sm_scale,
                                    self.max_seq_len, self.out, seq_lens_out=self.lens1)

    def make_fp8(self, k_scale: float = 0.03, v_scale: float = 0.03):
        """fp8 (E4M3) copies of the pools (aliased prefix pages hold the same codes) and the scratch of the group call"""
        from paper_2512_22560_b200 import rollart
        b, spec = self.batch, self.spec
        self.k8 = (b.k_pool.float() * (1.0 / k_scale)).to(torch.float8_e4m3fn).view(torch.uint8)
        self.v8 = (b.v_pool.float() * (1.0 / v_scale)).to(torch.float8_e4m3fn).view(torch.uint8)
        self.ks, self.vs = k_scale, v_scale
        need = rollart.obs_chunk_fp8_scratch_size(self.group_indptr.numel() - 1, spec.num_kv_heads, spec.page_size, self.max_seq_len)
        self.scratch = torch.empty(need, dtype=torch.uint8, device=self.device)

    def step_group_fp8(self):
        b = self.batch
        self.ctx.kv_append_fp8(self.k8, self.v8, self.table, self.lens0, self.new_indptr, b.k_new, b.v_new, self.ks, self.vs,
                               seq_lens_out=self.lens1)
        self.ctx.group_decode_attn_fp8(self.k8, self.v8, self.table, self.lens1, self.group_indptr, self.shared, self.q,
                                       self.spec.sm_scale, self.ks, self.vs, self.max_seq_len, self.out, self.scratch)

    def step_plain_fp8(self):
        b = self.batch
        self.ctx.append_decode_attn_fp8(self.k8, self.v8, self.table, self.lens0, b.k_new, b.v_new, self.q, self.spec.sm_scale,
                                        self.ks, self.vs, self.max_seq_len, self.out, seq_lens_out=self.lens1)

    def time(self, fn, steps: int, warmup: int) -> float:
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize(self.device)
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(steps):
            fn()
        t1.record()
        torch.cuda.synchronize(self.device)
        self.ctx.check()
        return t0.elapsed_time(t1) / steps


def chunk_flops(spec: W.WorkloadSpec, lens_after: np.ndarray, n_new: np.ndarray) -> float:
    """Causal-exact flops of the chunk call: every (row, visible key) pair costs 4*D per q head (QK^T and PV)."""
    pairs = 0
    for L, n in zip(lens_after.astype(np.int64), n_new.astype(np.int64)):
        prior = L - n
        pairs += n * prior + n * (n + 1) // 2
    return float(pairs) * spec.num_q_heads * 4 * spec.head_dim


class ChunkWorkload:
    """The observation-chunk half of a mixed batch: bulk append of the chunks, then chunk attention."""

    def __init__(self, spec: W.WorkloadSpec, seed: int, device: torch.device):
        from paper_2512_22560_b200 import rollart
        self.spec, self.device = spec, device
        b = W.make_batch(spec, seed=seed, device=device)
        self.batch = b
        ids = b.chunk_ids
        rows, q_indptr = b.chunk_rows()
        i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
        ridx = torch.from_numpy(rows).to(device)
        self.table, self.lens0, self.lens1 = i32(b.page_table), i32(b.seq_lens_before), i32(b.seq_lens_after)
        self.traj_ids, self.q_indptr = i32(ids), i32(q_indptr)
        self.q = b.q_new[ridx].contiguous()
        self.k_new, self.v_new = b.k_new[ridx].contiguous(), b.v_new[ridx].contiguous()
        self.out = torch.empty_like(self.q)
        self.max_seq_len = int(b.seq_lens_after.max())
        self.ctx = rollart.Context(device.index or 0, rollart.workspace_size(len(ids), spec.num_q_heads, spec.num_kv_heads,
                                                                            self.max_seq_len))
        self.flops = chunk_flops(spec, b.seq_lens_after[ids], b.n_new[ids])
        self.append_bytes = 2 * 2 * self.k_new.numel() * 2      # K and V rows, read + write
        self.rows = int(self.q.shape[0])

    def append(self):
        self.ctx.kv_append(self.batch.k_pool, self.batch.v_pool, self.table, self.lens0, self.q_indptr, self.k_new, self.v_new,
                           traj_ids=self.traj_ids, seq_lens_out=self.lens1)

    def attend(self):
        self.ctx.obs_chunk_attn(self.batch.k_pool, self.batch.v_pool, self.table, self.lens1, self.q_indptr, self.q,
                                self.spec.sm_scale, self.max_seq_len, self.out, traj_ids=self.traj_ids)

    def time(self, steps: int, warmup: int):
        for _ in range(warmup):
            self.append(); self.attend()
        torch.cuda.synchronize(self.device)
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
        for s in range(steps):
            ev[s][0].record(); self.append(); ev[s][1].record(); self.attend(); ev[s][2].record()
        torch.cuda.synchronize(self.device)
        self.ctx.check()
        return (float(np.mean([e[0].elapsed_time(e[1]) for e in ev])), float(np.mean([e[1].elapsed_time(e[2]) for e in ev])))


    def time_fp8(self, steps: int, warmup: int, k_scale: float = 0.03, v_scale: float = 0.03):
        """The same half over fp8 (E4M3) pools: quantising append of the chunks, then chunk attention over the fp8 cache
        (expansion of the listed contexts to bf16 into a scratch pool + the bf16 kernel).  (append ms, attention ms)"""
        from paper_2512_22560_b200 import rollart
        b, spec = self.batch, self.spec
        k8 = (b.k_pool.float() * (1.0 / k_scale)).to(torch.float8_e4m3fn).view(torch.uint8)
        v8 = (b.v_pool.float() * (1.0 / v_scale)).to(torch.float8_e4m3fn).view(torch.uint8)
        ids = b.chunk_ids
        pages = int(((b.seq_lens_after[ids].astype(np.int64) + spec.page_size - 1) // spec.page_size).sum())
        need = rollart.obs_chunk_fp8_scratch_size(len(ids), spec.num_kv_heads, spec.page_size, self.max_seq_len, total_pages=pages)
        scratch = torch.empty(need, dtype=torch.uint8, device=self.device)

        def append():
            self.ctx.kv_append_fp8(k8, v8, self.table, self.lens0, self.q_indptr, self.k_new, self.v_new, k_scale, v_scale,
                                   traj_ids=self.traj_ids, seq_lens_out=self.lens1)

        def attend():
            self.ctx.obs_chunk_attn_fp8(k8, v8, self.table, self.lens1, self.q_indptr, self.q, spec.sm_scale, k_scale, v_scale,
                                        self.max_seq_len, self.out, scratch, traj_ids=self.traj_ids)

        for _ in range(warmup):
            append(); attend()
        torch.cuda.synchronize(self.device)
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
        for i in range(steps):
            ev[i][0].record(); append(); ev[i][1].record(); attend(); ev[i][2].record()
        torch.cuda.synchronize(self.device)
        self.ctx.check()
        return (float(np.mean([e[0].elapsed_time(e[1]) for e in ev])), float(np.mean([e[1].elapsed_time(e[2]) for e in ev])),
                need)


class CpuBaseline:
    """The oracle, as it stands, timed on a bounded sample of the workload's trajectories."""

    def __init__(self, spec: W.WorkloadSpec, seed: int, budget_s: float = 15.0):
        import oracle
        self.oracle = oracle
        self.spec = spec
        layout = W.make_layout(spec, seed=seed)
        dec = layout.decode_ids
        cand = np.random.default_rng(seed).permutation(dec)
        # tensors for a bounded prefix of the candidates (at most 1M context tokens on the host)
        keep, toks = [], 0
        for t in cand:
            if keep and toks + int(layout.seq_lens_before[t]) > (1 << 20):
                break
            keep.append(int(t))
            toks += int(layout.seq_lens_before[t])
        self.full = _sample_tensors(layout, keep)
        self.n_dec = len(dec)
        t_cal, tok_cal = self.run([0])
        per_tok = t_cal / max(1, tok_cal)
        take, acc = [], 0.0
        for i in range(len(keep)):
            cost = per_tok * int(self.full.seq_lens_before[i] + 1)
            if take and acc + cost > budget_s:
                break
            take.append(i)
            acc += cost
        self.take = take

    def run(self, ids):
        sub = W.extract_trajs(self.full, ids)
        kp, vp = W.bf16_to_u16(sub.k_pool), W.bf16_to_u16(sub.v_pool)
        k_new, v_new = W.bf16_to_u16(sub.k_new), W.bf16_to_u16(sub.v_new)
        rows = sub.decode_rows(np.arange(len(ids)))
        q = W.bf16_to_u16(sub.q_new[rows])
        t0 = time.perf_counter()
        after = self.oracle.kv_append(kp, vp, sub.page_table, sub.seq_lens_before, sub.new_indptr, k_new, v_new)
        self.oracle.decode_attn(kp, vp, sub.page_table, after, q, self.spec.sm_scale)
        return time.perf_counter() - t0, int(after.sum())

    def measure(self):
        t, toks = self.run(self.take)
        # a sample that finishes in a fraction of a second is repeated (fresh copies of the pools each pass) until
        # about 1.5 s of wall time on all cores has gone by; the mean pass is reported
        passes = [t]
        while sum(passes) < 1.5 and len(passes) < 30:
            passes.append(self.run(self.take)[0])
        t = float(np.mean(passes))
        info = {"value": len(self.take) / t, "unit": UNIT, "cores": self.oracle.num_threads(), "kind": "oracle",
                "sample": f"{len(self.take)} of {self.n_dec} trajectories of {self.spec.name} ({toks} context tokens), "
                          f"append + decode, mean of {len(passes)} passes of {t:.2f} s wall"}
        return info, t, len(self.take)


def _sample_tensors(layout: W.Batch, ids) -> W.Batch:
    """CPU tensors for trajectories `ids` only (compact pool), same distributions as the full recipe."""
    spec = layout.spec
    P = spec.page_size
    ids = np.asarray(ids, dtype=np.int64)
    import dataclasses
    sub = dataclasses.replace(spec, num_traj=len(ids), name=spec.name + "_cpu_sample")
    lens = layout.seq_lens_before[ids].copy()
    n_new = layout.n_new[ids].copy()
    pages = (lens.astype(np.int64) + n_new + P - 1) // P
    table, num_pages = W.build_page_table(pages, spec.spare_pages, np.random.default_rng(layout.seed + 1))
    indptr = np.zeros(len(ids) + 1, dtype=np.int32)
    indptr[1:] = np.cumsum(n_new)
    b = W.Batch(sub, layout.seed, lens, n_new, layout.is_chunk[ids].copy(), indptr, table, num_pages)
    return W.fill_tensors(b, "cpu")


def rank_seed(seed: int, rank: int) -> int:
    """Replicas own disjoint, independently drawn trajectories: one seed per rank."""
    return seed + rank


def reduce_over_ranks(dist, device, maxima, sums):
    """Max over ranks of the timings and sum over ranks of the unit counts (identity when dist is None)."""
    t = torch.tensor(list(maxima), dtype=torch.float64, device=device)
    u = torch.tensor(list(sums), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return t.tolist(), u.tolist()


# ---- KV hand-off between two workers (Sec. 6.3: with prefill/decode disaggregation a trajectory's cache moves to another
# worker; Sec. 6.1: a trajectory resumes elsewhere).  Sender: rollart_kv_gather into contiguous rows; the rows cross to the
# receiver's own buffer (torch.distributed send / recv: NCCL between GPUs, no peer pointer is handed to any kernel);
# receiver: rollart_pages_reserve + rollart_kv_append onto its own pages.

def handoff_plan(lens):
    """indptr of the contiguous hand-off buffer for trajectories of these lengths (int32 [n + 1])"""
    indptr = np.concatenate([[0], np.cumsum(np.asarray(lens, dtype=np.int64))])
    if indptr[-1] >= 2 ** 31:
        raise ValueError("too many rows for one hand-off")
    return indptr.astype(np.int32)


def handoff_bytes(total_rows: int, num_kv_heads: int, head_dim: int, elem_bytes: int = 2) -> int:
    """bytes that cross between the workers: K and V rows"""
    return 2 * int(total_rows) * num_kv_heads * head_dim * elem_bytes


def handoff_send(dist, dst: int, lens, k_rows: torch.Tensor, v_rows: torch.Tensor) -> int:
    """Sender side: the lengths first (the receiver sizes its buffers from them), then the K and the V rows."""
    dev = k_rows.device
    lens_t = torch.as_tensor(np.asarray(lens, dtype=np.int32), device=dev)
    dist.send(torch.tensor([lens_t.numel()], dtype=torch.int32, device=dev), dst)
    dist.send(lens_t, dst)
    dist.send(k_rows, dst)
    dist.send(v_rows, dst)
    return k_rows.numel() * k_rows.element_size() + v_rows.numel() * v_rows.element_size()


def handoff_recv(dist, src: int, device, num_kv_heads: int, head_dim: int, dtype=torch.bfloat16):
    """Receiver side: (lens, indptr, k_rows, v_rows) in the receiver's own memory."""
    n = torch.zeros(1, dtype=torch.int32, device=device)
    dist.recv(n, src)
    lens_t = torch.zeros(int(n.item()), dtype=torch.int32, device=device)
    dist.recv(lens_t, src)
    lens = lens_t.cpu().numpy()
    indptr = handoff_plan(lens)
    k_rows = torch.empty(int(indptr[-1]), num_kv_heads, head_dim, dtype=dtype, device=device)
    v_rows = torch.empty_like(k_rows)
    dist.recv(k_rows, src)
    dist.recv(v_rows, src)
    return lens, indptr, k_rows, v_rows


def run_handoff(args, dist, rank: int, world: int, device):
    """`--handoff`: world size 2 = sender (rank 0) and receiver (rank 1); world size 1 = both roles on one GPU with the
    transfer left out (a check of everything but the wire).  The received cache must serve a decode call with the
    sender's bits."""
    from paper_2512_22560_b200 import rollart
    spec = W.CONFIGS[args.config]
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    times, moved, check = {}, 0, None
    k_rows = v_rows = lens = indptr = q = ref_out = None
    if rank == 0:
        b = W.make_batch(spec, seed=args.seed, device=device)
        lens = b.seq_lens_before
        indptr = handoff_plan(lens)
        table, d_lens = i32(b.page_table), i32(lens)
        ctx = rollart.Context(device.index or 0, rollart.workspace_size(spec.num_traj, spec.num_q_heads, spec.num_kv_heads, int(lens.max())))
        k_rows = torch.empty(int(indptr[-1]), spec.num_kv_heads, spec.head_dim, dtype=torch.bfloat16, device=device)
        v_rows = torch.empty_like(k_rows)
        a, z = ev(), ev()
        ctx.kv_gather(b.k_pool, b.v_pool, table, d_lens, i32(indptr), k_rows, v_rows)          # warm-up
        a.record()
        ctx.kv_gather(b.k_pool, b.v_pool, table, d_lens, i32(indptr), k_rows, v_rows)
        z.record()
        q = b.q_new[torch.from_numpy(b.decode_rows(np.arange(spec.num_traj))).to(device)].contiguous()
        ref_out = torch.empty_like(q)
        ctx.decode_attn(b.k_pool, b.v_pool, table, d_lens, q, spec.sm_scale, int(lens.max()), ref_out)
        ctx.check()
        times["gather_ms"] = a.elapsed_time(z)
        if world == 2:
            torch.cuda.synchronize(device)
            t0 = time.perf_counter()
            moved = handoff_send(dist, 1, lens, k_rows, v_rows)
            dist.send(q, 1)
            dist.send(ref_out, 1)
            torch.cuda.synchronize(device)
            times["transfer_ms"] = (time.perf_counter() - t0) * 1e3
        ctx.close()
        del b
    if rank == world - 1:
        if world == 2:
            torch.cuda.synchronize(device)
            t0 = time.perf_counter()
            lens, indptr, k_rows, v_rows = handoff_recv(dist, 0, device, spec.num_kv_heads, spec.head_dim)
            torch.cuda.synchronize(device)
            times["transfer_ms"] = (time.perf_counter() - t0) * 1e3
            q = torch.empty(len(lens), spec.num_q_heads, spec.head_dim, dtype=torch.bfloat16, device=device)
            ref_out = torch.empty_like(q)
            dist.recv(q, 0)
            dist.recv(ref_out, 0)
        # the receiver's own pool and bookkeeping: every page free, every row empty
        P = spec.page_size
        pages = (np.asarray(lens, dtype=np.int64) + P - 1) // P
        num_pages, max_pages, T = int(pages.sum()) + 8, int(pages.max()), len(lens)
        k_pool = torch.zeros(num_pages, spec.num_kv_heads, P, spec.head_dim, dtype=torch.bfloat16, device=device)
        v_pool = torch.zeros_like(k_pool)
        free = torch.arange(num_pages, dtype=torch.int32, device=device)
        cnt = torch.tensor([num_pages], dtype=torch.int32, device=device)
        table = torch.full((T, max_pages), -1, dtype=torch.int32, device=device)
        lens0, lens1 = torch.zeros(T, dtype=torch.int32, device=device), torch.zeros(T, dtype=torch.int32, device=device)
        ctx = rollart.Context(device.index or 0, rollart.workspace_size(T, spec.num_q_heads, spec.num_kv_heads, int(max(lens))))
        a, z = ev(), ev()
        a.record()
        ctx.pages_reserve(free, cnt, P, table, lens0, i32(lens))
        ctx.kv_append(k_pool, v_pool, table, lens0, i32(indptr), k_rows, v_rows, seq_lens_out=lens1)
        z.record()
        out = torch.empty_like(q)
        ctx.decode_attn(k_pool, v_pool, table, lens1, q, spec.sm_scale, int(max(lens)), out)
        ctx.check()
        times["reserve_append_ms"] = a.elapsed_time(z)
        check = bool(torch.equal(out.view(torch.int16), ref_out.view(torch.int16)))
        ctx.close()
    keys = ["gather_ms", "transfer_ms", "reserve_append_ms"]
    (t_max), _ = reduce_over_ranks(dist, device, [times.get(k, 0.0) for k in keys], [0])
    ok = torch.tensor([1.0 if check in (None, True) else 0.0], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(ok, op=dist.ReduceOp.MIN)
    if rank == 0:
        total_rows = int(indptr[-1])
        nbytes = handoff_bytes(total_rows, spec.num_kv_heads, spec.head_dim)
        line = {"workload": spec.name + " (KV hand-off: gather -> transfer -> reserve + append)", "n_gpus": world,
                "trajectories": int(len(lens)), "rows": total_rows, "bytes_moved": nbytes if world == 2 else 0,
                "decode_over_received_cache_bit_identical": bool(ok.item() == 1.0)}
        line.update({k: v for k, v in zip(keys, t_max)})
        if world == 2 and t_max[1] > 0:
            line["transfer_gbs"] = nbytes / (t_max[1] * 1e-3) / 1e9
        else:
            line["note"] = "one GPU: sender and receiver roles on the same device, no transfer"
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def run_reference(args):
    """`--impl reference`: the CPU oracle on a bounded sample per step (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    spec = W.CONFIGS[args.config]
    times, n = [], 0
    info = None
    base = CpuBaseline(spec, args.seed, budget_s=args.ref_budget)
    for s in range(args.warmup + args.steps):
        info, t, n = base.measure()
        if s >= args.warmup:
            times.append(t)
    ms = 1e3 * float(np.mean(times))
    value = n / (ms / 1e3)
    info["value"] = value
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "impl": "reference",
            "config": {"workload": spec.name, "note": "CPU fp64 oracle on a bounded sample of the workload per step"},
            "cpu_baseline": info,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1, help="index into the five workload recipes (headline: 1)")
    ap.add_argument("--seed", type=int, default=W.MASTER_SEED)
    ap.add_argument("--ref-budget", type=float, default=12.0, help="seconds of oracle work per reference step")
    ap.add_argument("--no-extra", action="store_true", help="skip the other decode workloads and the CPU baseline")
    ap.add_argument("--chunk", action="store_true", help="time only the observation-chunk half of --config (for profiling)")
    ap.add_argument("--shrink", type=int, default=1, help="with --chunk: divide context lengths by this (small profiling case)")
    ap.add_argument("--fp8", action="store_true", help="time only the fp8-pool decode step of --config (for profiling)")
    ap.add_argument("--handoff", action="store_true", help="KV hand-off between two workers (--gpus 2) or both roles on one GPU")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    if args.impl == "reference":
        return run_reference(args)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=device)

    spec = W.CONFIGS[args.config]
    if args.handoff:
        if world > 2:
            raise SystemExit("--handoff runs on 1 or 2 GPUs")
        return run_handoff(args, dist, rank, world, device)
    if args.chunk:
        if args.shrink > 1:
            spec = W.shrink(spec, max(2, spec.num_traj // args.shrink), args.shrink)
        cw = ChunkWorkload(spec, args.seed, device)
        app_ms, att_ms = cw.time(args.steps, args.warmup)
        print(json.dumps({"workload": spec.name + " (chunk half)", "chunk_rows": cw.rows, "chunk_attn_ms": att_ms,
                          "tflops": cw.flops / (att_ms * 1e-3) / 1e12, "append_ms": app_ms,
                          "append_gbs": cw.append_bytes / (app_ms * 1e-3) / 1e9}))
        return 0
    if args.fp8:
        w8 = DecodeWorkload(spec, args.seed, device)
        f8_ms, f8_bytes = w8.time_fp8_steps(args.steps, args.warmup)
        print(json.dumps({"workload": spec.name + " (fp8 pools: fused quantised append + decode)", "step_ms": f8_ms,
                          "decode_tokens_per_s": w8.n_items / (f8_ms * 1e-3), "hbm_gbs_of_fp8_bytes": f8_bytes / (f8_ms * 1e-3) / 1e9}))
        return 0
    wl = DecodeWorkload(spec, rank_seed(args.seed, rank), device)      # replicas: each rank owns its own trajectories

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(device)

    barrier()
    with ClockSampler(local) as clocks:
        # loops of exactly --steps steps; short loops are repeated until the timed region spans about a quarter of a
        # second, so that the value does not rest on one window of a few milliseconds and the clock sampler sees it
        loop_ms = wl.time_steps(args.steps, args.warmup, min_total_ms=250.0)
    barrier()
    per_step = np.array(loop_ms) / args.steps
    launches = args.steps * len(loop_ms)          # one kernel launch per step (rollart_append_decode_attn)
    # the host-driven loop needs a longer warm-up than the device-timed one: its first few hundred steps run
    # up to 25 % slower (host-side caches and clocks), which 3 steps do not cover
    e2e_steps = max(10, min(200, max(args.steps, 200) // 4))     # per loop; five loops, the median is reported
    e2e_ms, h2d, d2h = wl.time_e2e(e2e_steps, max(args.warmup, 200))

    (ms_per_step, ms_min, ms_max, e2e_ms_step), (n_items_all,) = reduce_over_ranks(
        dist, device, [float(np.median(per_step)), float(per_step.min()), float(per_step.max()), e2e_ms / e2e_steps], [wl.n_items])
    dec_ms = ms_per_step

    if rank == 0:
        peak, peak_kind = measured_peaks()
        achieved = wl.bytes / (dec_ms * 1e-3) / 1e9
        main = {
            "metric": METRIC, "value": n_items_all / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "repeats": len(loop_ms), "ms_per_step_min": ms_min, "ms_per_step_median": ms_per_step, "ms_per_step_max": ms_max,
            "config": {"workload": spec.name, "trajectories_per_gpu": wl.n_items, "num_q_heads": spec.num_q_heads,
                       "num_kv_heads": spec.num_kv_heads, "page_size": spec.page_size,
                       "context_tokens_per_gpu": int(wl.lens_after_host.sum()),
                       "step": "rollart_append_decode_attn: KV append of 1 token/trajectory + decode attention (split-KV partials, last-arriver LSE combine) in one launch, one attention layer",
                       "l2": "inputs larger than L2: %.2f GB of KV read per step" % (wl.bytes / 1e9),
                       "timing": "loops of exactly `steps` steps between two CUDA events, repeated `repeats` times back to back; ms_per_step = median loop / steps, max over ranks",
                       "parallelism": f"replicas x{world} (independent trajectories, no collective)"},
            "hbm_gbs": achieved, "hbm_frac_of_nominal_8tbs": achieved / NOMINAL_HBM_GBS,
            "e2e": {"value": n_items_all / (e2e_ms_step * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms_step,
                    "note": "per step one rollart_append_decode_attn_host call (arguments marshalled once): q, k_new, v_new host->device from one pinned buffer, out written by the kernel into a pinned host buffer, host sync; the KV pool is resident engine state; median of five loops"},
            "gpu_launches": int(launches),
            "clocks": clocks.summary(),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_kind": f"of {peak_kind}",
                         "traffic": measured_traffic(spec.name, args.seed),
                         "kernel": "decode_splitkv_kernel (append of the new token, partial attention and split combine in one launch)",
                         "algorithmic_bytes_per_launch": wl.bytes, "ms_per_launch": dec_ms},
        }
        targets = {spec.name: {"ms": dec_ms, "hbm_gbs": achieved, "frac_of_measured": achieved / peak,
                               "frac_of_nominal_8tbs": achieved / NOMINAL_HBM_GBS}}
        line = {}
        if not args.no_extra and world == 1:
            extra = {}
            del wl
            torch.cuda.empty_cache()
            for ci in (1, 2, 3):
                # the decode step over fp8 pools (half the KV bytes), beside the bf16 step of the same workload
                name = W.CONFIGS[ci].name + "_fp8_pool"
                try:
                    w8 = DecodeWorkload(W.CONFIGS[ci], args.seed, device)
                    bf_ms = float(np.median(w8.time_steps(200 if ci == 1 else 20, 3))) / (200 if ci == 1 else 20)
                    f8_ms, f8_bytes = w8.time_fp8_steps(200 if ci == 1 else 20, 3)
                    extra[name] = {"step_ms": f8_ms, "bf16_step_ms": bf_ms, "speedup_over_bf16_step": bf_ms / f8_ms,
                                   "decode_tokens_per_s": w8.n_items / (f8_ms * 1e-3),
                                   "hbm_gbs_of_fp8_bytes": f8_bytes / (f8_ms * 1e-3) / 1e9,
                                   "frac_of_measured": f8_bytes / (f8_ms * 1e-3) / 1e9 / peak,
                                   "launches_per_step": 1}
                    w8.ctx.close()
                    del w8
                    torch.cuda.empty_cache()
                except Exception as e:
                    extra[name] = {"error": repr(e)}
            try:
                # the tiny case lives in L2: a latency figure, back to back and after a write larger than L2
                w0 = DecodeWorkload(W.CONFIGS[0], args.seed, device)
                hot_ms = float(np.median(w0.time_steps(200, 10, min_total_ms=50.0))) / 200
                flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
                ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
                for a, b in ev:
                    flush.fill_(1)
                    a.record(); w0.step(); b.record()
                torch.cuda.synchronize(device)
                # 16 steps captured into one CUDA graph (Sec. 7.1: rollout runs with CUDA graphs): the launch period
                # without the host's issue rate in it
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=torch.cuda.Stream(device=device)):
                    for _ in range(16):
                        w0.step()
                for _ in range(3):
                    graph.replay()
                g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                g0.record()
                for _ in range(20):
                    graph.replay()
                g1.record()
                torch.cuda.synchronize(device)
                w0.ctx.check()
                extra[W.CONFIGS[0].name] = {"step_us_back_to_back": hot_ms * 1e3,
                                            "step_us_graph_replay": g0.elapsed_time(g1) / (20 * 16) * 1e3,
                                            "step_us_after_l2_flush": float(np.median([a.elapsed_time(b) for a, b in ev])) * 1e3,
                                            "trajectories": w0.n_items, "kv_bytes": w0.bytes,
                                            "note": "back to back = launch period of eager calls; graph replay = the same from a CUDA graph of "
                                                    "16 steps (no host issue cost); after flush = events around one launch"}
                w0.ctx.close()
                del w0, flush
                torch.cuda.empty_cache()
            except Exception as e:
                extra[W.CONFIGS[0].name] = {"error": repr(e)}
            for ci in (2, 3, 4):
                try:
                    w2 = DecodeWorkload(W.CONFIGS[ci], args.seed, device)
                    loops = np.array(w2.time_steps(20, 3, min_total_ms=150.0)) / 20
                    dms = float(np.median(loops))
                    gbs = w2.bytes / (dms * 1e-3) / 1e9
                    extra[W.CONFIGS[ci].name] = {"step_ms": dms, "step_ms_min": float(loops.min()), "step_ms_max": float(loops.max()),
                                                 "repeats": len(loops), "hbm_gbs": gbs,
                                                 "frac_of_measured": gbs / peak, "frac_of_nominal_8tbs": gbs / NOMINAL_HBM_GBS,
                                                 "decode_tokens_per_s": w2.n_items / (dms * 1e-3),
                                                 "trajectories": w2.n_items}
                    if ci in (2, 3):
                        targets[W.CONFIGS[ci].name] = {"ms": dms, "hbm_gbs": gbs, "frac_of_measured": gbs / peak,
                                                       "frac_of_nominal_8tbs": gbs / NOMINAL_HBM_GBS}
                    if ci == 3:
                        g_ms, g_bytes = w2.time_gather()
                        extra[W.CONFIGS[ci].name].update({"kv_gather_ms": g_ms, "kv_gather_gbs": g_bytes / (g_ms * 1e-3) / 1e9,
                                                          "kv_gather_frac_of_measured_hbm": g_bytes / (g_ms * 1e-3) / 1e9 / peak})
                    w2.ctx.close()
                    del w2
                    torch.cuda.empty_cache()
                except Exception as e:  # report, never hide
                    extra[W.CONFIGS[ci].name] = {"error": repr(e)}
            try:
                cw = ChunkWorkload(W.CONFIGS[4], args.seed, device)
                app_ms, att_ms = cw.time(5, 2)                     # five launches: the GPU is still near its top clock
                with ClockSampler(local) as chunk_clocks:          # twenty more: the leg now runs under the power cap
                    _, att_sus_ms = cw.time(20, 0)
                tf_peak, tf_burst = 1399.5, 1590.0           # the fallbacks (sustained, burst) if the measured peaks are absent
                try:
                    with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
                        mp = json.load(f)
                    tf_peak, tf_burst = float(mp["bf16_tflops_sustained"]), float(mp["bf16_tflops"])
                except Exception:
                    pass
                tfs = cw.flops / (att_ms * 1e-3) / 1e12
                extra["cfg4_mixed_multiturn_chunk_half"] = {
                    "chunk_rows": cw.rows, "chunk_attn_ms": att_ms, "tflops": tfs, "frac_of_measured_bf16_burst": tfs / tf_burst,
                    "chunk_attn_ms_sustained": att_sus_ms, "tflops_sustained": cw.flops / (att_sus_ms * 1e-3) / 1e12,
                    "frac_of_measured_bf16_sustained": cw.flops / (att_sus_ms * 1e-3) / 1e12 / tf_peak,
                    "note": "tflops: mean of 5 launches after 2 warm-ups, against the measured burst rate; tflops_sustained: mean of the 20 launches that follow, with the clocks sampled meanwhile, against the measured sustained rate",
                    "kernel": "chunk_attn_pair_kernel (tcgen05 cta_group::2, one launch per call)",
                    "clocks": chunk_clocks.summary(),
                    "append_ms": app_ms, "append_gbs": cw.append_bytes / (app_ms * 1e-3) / 1e9,
                    "append_frac_of_measured_hbm": cw.append_bytes / (app_ms * 1e-3) / 1e9 / peak}
                try:
                    a8, t8, need = cw.time_fp8(5, 2)
                    extra["cfg4_mixed_multiturn_chunk_half_fp8_pool"] = {
                        "chunk_attn_ms": t8, "bf16_chunk_attn_ms_sustained": att_sus_ms, "ratio_to_bf16": t8 / att_sus_ms,
                        "tflops": cw.flops / (t8 * 1e-3) / 1e12, "append_ms": a8, "scratch_bytes": need,
                        "launches": 4, "note": "contexts expanded to bf16 into the scratch pool (pages packed by a plan kernel), then the two bf16 kernels"}
                except Exception as e:
                    extra["cfg4_mixed_multiturn_chunk_half_fp8_pool"] = {"error": repr(e)}
                cw.ctx.close()
                del cw
                torch.cuda.empty_cache()
            except Exception as e:
                extra["cfg4_mixed_multiturn_chunk_half"] = {"error": repr(e)}
            try:
                rw = ChunkWorkload(W.RECOMPUTE, args.seed, device)
                app_ms, att_ms = rw.time(3, 2)
                rtf = rw.flops / (att_ms * 1e-3) / 1e12
                extra[W.RECOMPUTE.name] = {"rows": rw.rows, "chunk_attn_ms": att_ms, "tflops": rtf,
                                           "frac_of_measured_bf16_sustained": rtf / tf_peak, "frac_of_measured_bf16_burst": rtf / tf_burst,
                                           "append_ms": app_ms, "append_gbs": rw.append_bytes / (app_ms * 1e-3) / 1e9}
                rw.ctx.close()
                del rw
                torch.cuda.empty_cache()
            except Exception as e:
                extra[W.RECOMPUTE.name] = {"error": repr(e)}
            for frac in (W.GROUP_SHARED_FRACTION, 1.0):
                name = "%s_shared%.2f" % (W.GROUP_DECODE.name, frac)
                try:
                    gw = GroupDecodeWorkload(W.GROUP_DECODE, args.seed, device, W.GROUP_SIZE, frac)
                    g_ms = gw.time(gw.step_group, 20, 3)
                    p_ms = gw.time(gw.step_plain, 20, 3)
                    extra[name] = {
                        "trajectories": gw.n_items, "group_size": W.GROUP_SIZE, "shared_fraction_of_shortest_member": frac,
                        "group_step_ms": g_ms, "plain_step_ms": p_ms, "speedup_over_plain_step": p_ms / g_ms,
                        "decode_tokens_per_s": gw.n_items / (g_ms * 1e-3),
                        "bytes_per_trajectory_definition": gw.bytes_per_trajectory_definition,
                        "bytes_unique_pages": gw.bytes_unique, "unique_gbs": gw.bytes_unique / (g_ms * 1e-3) / 1e9,
                        "plain_gbs": gw.bytes_per_trajectory_definition / (p_ms * 1e-3) / 1e9}
                    try:
                        gw.make_fp8()
                        g8 = gw.time(gw.step_group_fp8, 20, 3)
                        p8 = gw.time(gw.step_plain_fp8, 20, 3)
                        extra[name]["fp8_pool"] = {"group_step_ms": g8, "plain_step_ms": p8, "speedup_over_plain_fp8_step": p8 / g8,
                                                   "speedup_over_plain_bf16_step": p_ms / g8, "launches_per_group_step": 7}
                    except Exception as e:
                        extra[name]["fp8_pool"] = {"error": repr(e)}
                    gw.ctx.close()
                    del gw
                    torch.cuda.empty_cache()
                except Exception as e:
                    extra[name] = {"error": repr(e)}
            line["other_workloads"] = extra
            info, _, _ = CpuBaseline(spec, args.seed).measure()
            main["cpu_baseline"] = info
        # the long block of other workloads goes first, the headline keys and the three target workloads last
        line.update(main)
        line["targets"] = targets
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
