// Internal declarations shared by the translation units of librollart (not part of the ABI).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "rollart.h"

namespace rollart {

constexpr int kHeadDim = 128;
constexpr int kMaxGroup = 16;      // query heads per kv head
constexpr int kRowBytes = kHeadDim * 2;

// Device status word: 0 = ok, else the first rollart_status a kernel recorded.
// status[1] carries a detail value (the offending index) for the error text.
struct DeviceStatus {
    int code;
    int detail;
    int where;
    int fatal;   // set with a timeout: blocks that have not started yet return at once
};

__device__ __forceinline__ void report(DeviceStatus *st, int code, int detail, int where) {
    if (atomicCAS(&st->code, 0, code) == 0) {
        st->detail = detail;
        st->where = where;
    }
}

// eight bf16 (one 16-byte piece of a row) -> eight E4M3 codes: code = nearest (ties to even, saturating at +-448) of
// x * inv_scale, the product rounded to fp32 first
__device__ __forceinline__ uint2 quantize8(const uint4 &v, float inv_scale) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t h[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w[i] << 16) * inv_scale, hi = __uint_as_float(w[i] & 0xffff0000u) * inv_scale;
        uint16_t p;
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(p) : "f"(hi), "f"(lo));    // first operand -> upper byte
        h[i] = p;
    }
    return make_uint2(h[0] | (h[1] << 16), h[2] | (h[3] << 16));
}

struct PoolView {
    const __nv_bfloat16 *k;
    const __nv_bfloat16 *v;
    int num_pages, page_size, num_kv_heads;
};

struct TrajView {
    const int32_t *page_table;
    const int32_t *seq_lens;
    int max_pages, num_traj;
};

// ---- launchers (each enqueues on `stream`, returns the cudaError of the launch, and adds the
//      number of kernels it launched to *launches) ----
cudaError_t launch_kv_append(const rollart_kv_pool &pool, const rollart_trajs &trajs, const int32_t *traj_ids,
                             const int32_t *new_indptr, int n_items, int total_new, const void *k_new,
                             const void *v_new, int32_t *seq_lens_out, DeviceStatus *status, cudaStream_t stream,
                             int64_t *launches, bool fp8 = false, float k_scale = 1.f, float v_scale = 1.f,
                             bool rows_are_codes = false);

cudaError_t launch_kv_gather(const rollart_kv_pool &pool, const rollart_trajs &trajs, const int32_t *traj_ids,
                             const int32_t *out_indptr, int n_items, int total_rows, void *k_out, void *v_out,
                             DeviceStatus *status, cudaStream_t stream, int64_t *launches, bool fp8 = false);

cudaError_t launch_pages(bool reserve, int32_t *free_pages, int32_t *free_count, int capacity, int page_size,
                         int32_t *page_table, int max_pages, int32_t *seq_lens, int num_traj, const int32_t *traj_ids,
                         const int32_t *new_tokens, int n_items, DeviceStatus *status, cudaStream_t stream, int64_t *launches);

cudaError_t launch_pages_evict(int32_t *free_pages, int32_t *free_count, int capacity, int page_size, int32_t *page_table,
                               int max_pages, int32_t *seq_lens, int num_traj, const int32_t *start_version,
                               int current_version, int alpha, int32_t *evicted_ids, int32_t *n_evicted, DeviceStatus *status,
                               cudaStream_t stream, int64_t *launches);

// Host-side cache of the TMA tensor maps describing the K and V pools (re-encoded when the pools change).
struct TmaCache {
    bool valid;
    const void *k;
    const void *v;
    int num_pages, hkv, page_size, four_d, fp8;
    alignas(64) unsigned char kmap[128];
    alignas(64) unsigned char vmap[128];
};

struct AttnCall {
    PoolView pool;
    TrajView trajs;
    const int32_t *traj_ids;  // nullable
    const int32_t *q_indptr;  // NULL for decode (one row per item)
    int n_items;
    int total_q;              // rows of q/out
    int max_seq_len;
    const __nv_bfloat16 *q;
    int num_q_heads;
    float sm_scale;
    __nv_bfloat16 *out;
    float *lse;               // nullable
    void *workspace;
    size_t workspace_bytes;
    DeviceStatus *status;
    int sm_count;
    TmaCache *tma;
    // fused append + decode (NULL otherwise): new K/V rows [n_items][num_kv_heads][128] and the lengths after
    const __nv_bfloat16 *k_new;
    const __nv_bfloat16 *v_new;
    int32_t *seq_lens_out;
    // group decode (all NULL otherwise)
    const int32_t *page_offset;   // decode: per item, pages of the table row to skip (the keys before them are not attended to)
    const int32_t *shared_lens;   // chunk: per item, every query row of the item sees exactly the first shared_lens[i] keys
    float *out_f32;               // when set the result rows are written here in fp32 instead of bf16 to `out`
    const int32_t *item_order;    // chunk: per batch of kChunkItemsPerLaunch items, the order in which blocks take them
    uint32_t *redo_bits;          // chunk: kChunkRedoBits bits of the context, the units a second pass has to take; 64 more bytes behind them
    // fp8 (E4M3) pools (decode and fused append + decode): keys are k_scale * code value, values v_scale * code value.
    // The chunk kernel reads bf16 only; it multiplies its result by v_scale (1 for bf16 pools).
    bool fp8;
    float k_scale, v_scale;
};

size_t decode_workspace_bytes(int max_items, int num_q_heads, int num_kv_heads, int max_seq_len, int sm_count);
// returns cudaSuccess, or cudaErrorInvalidValue with *too_small = true if the workspace cannot hold the call
cudaError_t launch_decode_attn(const AttnCall &c, cudaStream_t stream, int64_t *launches, bool *too_small);
// zeroes the bookkeeping at the head of the workspace after a device-side error
cudaError_t decode_reset_workspace(void *workspace, size_t bytes, cudaStream_t stream);
cudaError_t launch_chunk_attn(const AttnCall &c, cudaStream_t stream, int64_t *launches, bool *too_small);
// diagnostic: a bounded in-kernel wait that must run out (see rollart_selftest_bounded_wait)
cudaError_t launch_bounded_wait_selftest(DeviceStatus *status, cudaStream_t stream, int64_t *launches);
// the causal chunk call on CTA pairs (no shared-prefix mode, bf16 output): what launch_chunk_attn runs for such calls
// items base .. base + n - 1 of the call (at most kChunkItemsPerLaunch), c.redo_bits zeroed on the stream before
cudaError_t launch_chunk_attn_pair(const AttnCall &c, int base, int n, cudaStream_t stream, int64_t *launches);

// Observation-chunk attention over fp8 pools: the listed trajectories' contexts are expanded to bf16 into a scratch
// pool (item i owns pages i * pages_per_item ..), with a scratch page table and scratch lengths behind the two pools.
struct Fp8ChunkScratch {
    int pages_per_item;            // row length of the scratch page table
    long long capacity_pages;      // pages each of the two scratch pools can hold
    size_t off_k, off_v, off_table, off_lens, off_first, bytes;
};
// bytes for pools of `total_pages` pages (negative or above n_items * pages_per_item: that worst case) plus the small arrays
size_t fp8_chunk_scratch_bytes(int n_items, int num_kv_heads, int page_size, int max_seq_len, long long total_pages);
// how a buffer of scratch_bytes is divided; capacity_pages = 0 if it cannot hold even one page
Fp8ChunkScratch fp8_chunk_scratch_layout(int n_items, int num_kv_heads, int page_size, int max_seq_len, size_t scratch_bytes);
// lens_override (nullable): per item, expand only that many tokens instead of the trajectory's length
cudaError_t launch_fp8_pages_to_bf16(const rollart_kv_pool &pool, const rollart_trajs &trajs, const int32_t *traj_ids,
                                     const int32_t *lens_override, int n_items, int max_seq_len,
                                     const Fp8ChunkScratch &layout, void *scratch, DeviceStatus *status, cudaStream_t stream,
                                     int64_t *launches);

// items per launch of the chunk kernel (its per-item table lives in shared memory)
constexpr int kChunkItemsPerLaunch = 1024;
constexpr int kChunkRedoBits = 4096;      // bitmap of the units of a chunk launch that its second pass computes again

// Group decode helpers.  `prepare` derives, per group, the trajectory whose table row stands for the shared
// prefix and, per item, the pages to skip; it also checks that the members alias the same pages there.
cudaError_t launch_group_prepare(const TrajView &trajs, const int32_t *traj_ids, int n_items, const int32_t *group_indptr,
                                 const int32_t *shared_lens, int n_groups, int page_size, int32_t *group_traj,
                                 int32_t *item_page_offset, int32_t *group_order, DeviceStatus *status, cudaStream_t stream,
                                 int64_t *launches);
// out = softmax-weighted sum of the two partial results (weights from their log-sum-exps); lse optional
cudaError_t launch_group_merge(const float *part_a, const float *lse_a, const float *part_b, const float *lse_b,
                               long long rows, __nv_bfloat16 *out, float *lse, cudaStream_t stream, int64_t *launches);

}  // namespace rollart
