// Helpers of the group decode step (rollart_group_decode_attn).
//
// The paper trains with GRPO at a group size of 8 and runs its rollout engine with prefix caching
// (Sec. 7.1): the members of a group hold the same prompt tokens and their page-table rows alias the
// same physical pages there.  The group decode step reads those pages once per group instead of once
// per member: the shared prefix goes through the tensor-core chunk kernel with the members' query rows
// stacked into one M-tile, the private remainder through the split-KV decode kernel, and the two partial
// results of every (item, head) are merged here from their log-sum-exps.
#include "rollart_internal.cuh"

namespace rollart {
namespace {

constexpr int kPrepThreads = 128;

// One block per group.  Writes group_traj[gi] (the member whose table row stands for the prefix) and
// item_page_offset[i] for the members, and verifies what the caller promised: indptr is a partition of
// the items, the shared length is a whole number of pages and not beyond any member's length, and the
// members' table rows agree on the shared pages.
__global__ void __launch_bounds__(kPrepThreads)
group_prepare_kernel(const int32_t *__restrict__ page_table, const int32_t *__restrict__ seq_lens,
                     const int32_t *__restrict__ traj_ids, int n_items, const int32_t *__restrict__ group_indptr,
                     const int32_t *__restrict__ shared_lens, int n_groups, int page_size, int max_pages, int num_traj,
                     int32_t *__restrict__ group_traj, int32_t *__restrict__ item_page_offset,
                     int32_t *__restrict__ group_order, DeviceStatus *status) {
    const int gi = blockIdx.x;
    {
        // Rank of this group among the groups of its launch batch by shared length, longest first (ties by index): the
        // prefix pass takes the groups in that order, so the long ones do not start last.  Whatever the lengths are,
        // (length, index) is a total order, so the ranks of a batch are a permutation of it.
        __shared__ int s_cnt[kPrepThreads / 32];
        const int base = gi / kChunkItemsPerLaunch * kChunkItemsPerLaunch;
        const int n = min(kChunkItemsPerLaunch, n_groups - base);
        const int mine = __ldg(shared_lens + gi);
        int cnt = 0;
        for (int j = threadIdx.x; j < n; j += kPrepThreads) {
            const int v = __ldg(shared_lens + base + j);
            cnt += (v > mine || (v == mine && base + j < gi)) ? 1 : 0;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        if ((threadIdx.x & 31) == 0) s_cnt[threadIdx.x >> 5] = cnt;
        __syncthreads();
        if (threadIdx.x == 0) {
            int rank = 0;
            for (int w = 0; w < kPrepThreads / 32; ++w) rank += s_cnt[w];
            group_order[base + rank] = gi - base;
        }
    }
    const int a = __ldg(group_indptr + gi), b = __ldg(group_indptr + gi + 1);
    const int s_len = __ldg(shared_lens + gi);
    bool bad = a < 0 || b < a || b > n_items || (gi == 0 && a != 0) || (gi == n_groups - 1 && b != n_items);
    if (bad) {
        if (threadIdx.x == 0) { report(status, ROLLART_ERR_BOUNDS, gi, 7); group_traj[gi] = 0; }
        return;
    }
    if (s_len < 0 || s_len % page_size != 0 || s_len / page_size > max_pages) {
        if (threadIdx.x == 0) report(status, ROLLART_ERR_BOUNDS, s_len, 7);
        bad = true;
    }
    const int pages = bad ? 0 : s_len / page_size;
    int t0 = 0;
    if (a < b) {
        t0 = traj_ids ? __ldg(traj_ids + a) : a;
        if (t0 < 0 || t0 >= num_traj) {
            if (threadIdx.x == 0) report(status, ROLLART_ERR_BOUNDS, t0, 7);
            t0 = 0;
            bad = true;
        }
    }
    if (threadIdx.x == 0) group_traj[gi] = t0;
    for (int i = a + threadIdx.x; i < b; i += kPrepThreads) {
        const int t = traj_ids ? __ldg(traj_ids + i) : i;
        int off = pages;
        if (t < 0 || t >= num_traj) { report(status, ROLLART_ERR_BOUNDS, t, 7); off = 0; }
        else if (s_len > __ldg(seq_lens + t)) { report(status, ROLLART_ERR_BOUNDS, s_len, 7); off = 0; }
        item_page_offset[i] = bad ? 0 : off;
    }
    if (bad || b - a < 2 || pages == 0) return;
    const int32_t *row0 = page_table + static_cast<long long>(t0) * max_pages;
    // every thread keeps its pages of the first member's row and compares the other members' rows against them
    for (int lp0 = threadIdx.x; lp0 < pages; lp0 += kPrepThreads * 4) {
        int ref[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int lp = lp0 + k * kPrepThreads;
            ref[k] = lp < pages ? __ldg(row0 + lp) : 0;
        }
        for (int m = a + 1; m < b; ++m) {
            const int t = traj_ids ? __ldg(traj_ids + m) : m;
            if (t < 0 || t >= num_traj) continue;      // reported above
            const int32_t *row = page_table + static_cast<long long>(t) * max_pages;
            bool differ = false;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int lp = lp0 + k * kPrepThreads;
                if (lp < pages && __ldg(row + lp) != ref[k]) differ = true;
            }
            if (differ) report(status, ROLLART_ERR_BOUNDS, m, 7);   // this member does not alias the group's prefix pages
        }
    }
}

// One warp per (item, query head) row: 32 lanes x 4 values.
__global__ void __launch_bounds__(256)
group_merge_kernel(const float *__restrict__ part_a, const float *__restrict__ lse_a, const float *__restrict__ part_b,
                   const float *__restrict__ lse_b, long long rows, __nv_bfloat16 *__restrict__ out, float *__restrict__ lse) {
    const long long row = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int lane = threadIdx.x & 31;
    const float la = __ldg(lse_a + row), lb = __ldg(lse_b + row);
    const float m = fmaxf(la, lb);
    float wa = 0.f, wb = 0.f, total = -INFINITY;
    if (m != -INFINITY) {
        const float ea = expf(la - m), eb = expf(lb - m);      // exp(-inf) = 0 for an empty part
        const float inv = 1.f / (ea + eb);
        wa = ea * inv; wb = eb * inv;
        total = m + logf(ea + eb);
    }
    const float4 xa = __ldg(reinterpret_cast<const float4 *>(part_a + row * kHeadDim) + lane);
    const float4 xb = __ldg(reinterpret_cast<const float4 *>(part_b + row * kHeadDim) + lane);
    __nv_bfloat162 lo = __floats2bfloat162_rn(xa.x * wa + xb.x * wb, xa.y * wa + xb.y * wb);
    __nv_bfloat162 hi = __floats2bfloat162_rn(xa.z * wa + xb.z * wb, xa.w * wa + xb.w * wb);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t *>(&lo); packed.y = *reinterpret_cast<uint32_t *>(&hi);
    reinterpret_cast<uint2 *>(out + row * kHeadDim)[lane] = packed;
    if (lse != nullptr && lane == 0) lse[row] = total;
}

}  // namespace

cudaError_t launch_group_prepare(const TrajView &trajs, const int32_t *traj_ids, int n_items, const int32_t *group_indptr,
                                 const int32_t *shared_lens, int n_groups, int page_size, int32_t *group_traj,
                                 int32_t *item_page_offset, int32_t *group_order, DeviceStatus *status, cudaStream_t stream,
                                 int64_t *launches) {
    if (n_groups <= 0) return cudaSuccess;
    group_prepare_kernel<<<n_groups, kPrepThreads, 0, stream>>>(trajs.page_table, trajs.seq_lens, traj_ids, n_items,
                                                                group_indptr, shared_lens, n_groups, page_size,
                                                                trajs.max_pages, trajs.num_traj, group_traj,
                                                                item_page_offset, group_order, status);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_group_merge(const float *part_a, const float *lse_a, const float *part_b, const float *lse_b,
                               long long rows, __nv_bfloat16 *out, float *lse, cudaStream_t stream, int64_t *launches) {
    if (rows <= 0) return cudaSuccess;
    const long long blocks = (rows + 7) / 8;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
    group_merge_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(part_a, lse_a, part_b, lse_b, rows, out, lse);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace rollart
