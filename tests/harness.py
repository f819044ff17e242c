"""Shared by the GPU parity tests: run a seeded batch through the CUDA library and the CPU oracle."""
import numpy as np
import torch

import oracle
from paper_2512_22560_b200 import rollart
from paper_2512_22560_b200 import workloads as W

ATOL, RTOL = 1e-2, 2e-2          # attention outputs: |err| <= 1e-2 + 2e-2 |ref|
LSE_ATOL, LSE_RTOL = 1e-3, 1e-3


def dev_i32(a, device):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)


class DeviceBatch:
    """Device-side views of a workloads.Batch (moves CPU tensors to the device if needed)."""

    def __init__(self, batch: W.Batch, device):
        self.b = batch
        self.device = device
        self.k_pool = batch.k_pool.to(device)
        self.v_pool = batch.v_pool.to(device)
        self.q_new = batch.q_new.to(device)
        self.k_new = batch.k_new.to(device)
        self.v_new = batch.v_new.to(device)
        self.page_table = dev_i32(batch.page_table, device)
        self.lens_before = dev_i32(batch.seq_lens_before, device)
        self.new_indptr = dev_i32(batch.new_indptr, device)
        self.lens_after = torch.full_like(self.lens_before, -7)

    def append(self, ctx: rollart.Context):
        ctx.kv_append(self.k_pool, self.v_pool, self.page_table, self.lens_before, self.new_indptr, self.k_new,
                      self.v_new, seq_lens_out=self.lens_after)


def make_ctx(spec, n_items, max_seq_len, device=0):
    return rollart.Context(device, rollart.workspace_size(max(1, n_items), spec.num_q_heads, spec.num_kv_heads, max_seq_len))


def oracle_append(batch: W.Batch):
    kp, vp = W.bf16_to_u16(batch.k_pool), W.bf16_to_u16(batch.v_pool)
    after = oracle.kv_append(kp, vp, batch.page_table, batch.seq_lens_before, batch.new_indptr,
                             W.bf16_to_u16(batch.k_new), W.bf16_to_u16(batch.v_new))
    return kp, vp, after


def error_stats(got: torch.Tensor, ref: np.ndarray):
    g = got.detach().float().cpu().numpy().astype(np.float64)
    err = np.abs(g - ref)
    rms_ref = float(np.sqrt(np.mean(ref ** 2))) if ref.size else 0.0
    return {
        "max_abs": float(err.max()) if err.size else 0.0,
        "rms": float(np.sqrt(np.mean(err ** 2))) if err.size else 0.0,
        "rms_ref": rms_ref,
        "worst_margin": float((err - (ATOL + RTOL * np.abs(ref))).max()) if err.size else -1.0,
    }


def assert_attn_close(got: torch.Tensor, ref: np.ndarray, what=""):
    assert tuple(got.shape) == ref.shape, (got.shape, ref.shape)
    st = error_stats(got, ref)
    assert np.isfinite(st["max_abs"]), f"{what}: non-finite output"
    assert st["worst_margin"] <= 0.0, f"{what}: outside |err| <= 1e-2 + 2e-2|ref|: {st}"
    # bf16 output rounding alone gives a relative RMS error near 2^-9; a wrong key or a dropped
    # tile shows up far above this bound even when the absolute tolerance would let it through
    assert st["rms"] <= 2.0 ** -7 * max(st["rms_ref"], 1e-3), f"{what}: rms error too large: {st}"
    return st


def assert_lse_close(got: torch.Tensor, ref: np.ndarray, what=""):
    g = got.detach().cpu().numpy().astype(np.float64)
    fin = np.isfinite(ref)
    assert np.array_equal(np.isneginf(g), np.isneginf(ref)), f"{what}: -inf pattern differs"
    err = np.abs(g[fin] - ref[fin])
    assert np.all(err <= LSE_ATOL + LSE_RTOL * np.abs(ref[fin])), f"{what}: lse max err {err.max()}"
