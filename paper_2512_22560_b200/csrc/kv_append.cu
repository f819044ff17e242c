// KV append: scatter the new tokens' K/V rows into the trajectories' pages (bit copy), and its
// inverse, KV gather: copy a trajectory's tokens from its pages into contiguous rows.
//
// One thread moves 16 bytes of a K row and the matching 16 bytes of the V row.  A (token, kv head)
// row is 256 B, so 16 consecutive threads cover it and a warp covers two heads of one token;
// both the source ([token][head][d]) and each destination row are contiguous, so every 16-lane
// group reads and writes one fully used 256 B segment.  The kernel is bound by HBM traffic for
// observation chunks and by launch latency for single decode tokens.
#include "rollart_internal.cuh"

namespace rollart {

namespace {

constexpr int kThreads = 256;
constexpr int kVecPerRow = kRowBytes / 16;  // 16 for a bf16 row (256 B), half as many for a row of 8-bit codes

// what an append does with a row: bit copy of bf16, bf16 quantised to E4M3 codes, or bit copy of E4M3 codes
enum AppendMode { kCopyBf16 = 0, kQuantize = 1, kCopyCodes = 2 };

// item whose row range [indptr[i], indptr[i+1]) holds `row`; indptr is non-decreasing
__device__ __forceinline__ int find_item(const int32_t *__restrict__ indptr, int n_items, int row) {
    int lo = 0, hi = n_items;  // invariant: indptr[lo] <= row < indptr[hi]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (__ldg(indptr + mid) <= row) lo = mid; else hi = mid;
    }
    return lo;
}

// kQuantize: the pools hold E4M3 codes (rows of 128 B); the new rows arrive as bf16 and are quantised on the way.
// kCopyCodes: pools and new rows both hold codes (a cache handed over by another worker); rows of 128 B, 8 threads each.
template <int kMode>
__global__ void __launch_bounds__(kThreads)
kv_append_kernel(void *__restrict__ k_pool, void *__restrict__ v_pool, float k_inv_scale, float v_inv_scale, int num_pages, int page_size,
                 int num_kv_heads, const int32_t *__restrict__ page_table, int max_pages,
                 const int32_t *__restrict__ seq_lens, int num_traj, const int32_t *__restrict__ traj_ids,
                 const int32_t *__restrict__ new_indptr, int n_items, int total_new,
                 const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new, int32_t *__restrict__ seq_lens_out,
                 DeviceStatus *status) {
    const long long gid = static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x;

    // lengths after the append, one thread per item
    if (seq_lens_out != nullptr && gid < n_items) {
        const int i = static_cast<int>(gid);
        const int t = traj_ids ? __ldg(traj_ids + i) : i;
        if (t < 0 || t >= num_traj) {
            report(status, ROLLART_ERR_BOUNDS, t, 1);
        } else {
            const int n = __ldg(new_indptr + i + 1) - __ldg(new_indptr + i);
            seq_lens_out[t] = __ldg(seq_lens + t) + n;
        }
    }

    constexpr int kVec = kMode == kCopyCodes ? kVecPerRow / 2 : kVecPerRow;   // 16-byte pieces of a source row
    const long long n_vec = static_cast<long long>(total_new) * num_kv_heads * kVec;
    if (gid >= n_vec) return;
    // the rows to move do not depend on where they go: start their loads before the chain of dependent
    // look-ups (item search, length, page id), so that the two latencies overlap
    const uint4 kv = __ldg(k_new + gid);
    const uint4 vv = __ldg(v_new + gid);
    const int c = static_cast<int>(gid % kVec);
    const long long rh = gid / kVec;
    const int h = static_cast<int>(rh % num_kv_heads);
    const int row = static_cast<int>(rh / num_kv_heads);

    const int i = find_item(new_indptr, n_items, row);
    const int t = traj_ids ? __ldg(traj_ids + i) : i;
    if (t < 0 || t >= num_traj) { report(status, ROLLART_ERR_BOUNDS, t, 1); return; }
    const int len = __ldg(seq_lens + t);
    if (len < 0) { report(status, ROLLART_ERR_BOUNDS, len, 1); return; }
    // a row outside its item's range means new_indptr is not a non-decreasing array from 0 to total_new
    const int first = __ldg(new_indptr + i);
    if (row < first || row >= __ldg(new_indptr + i + 1)) { report(status, ROLLART_ERR_BOUNDS, row, 1); return; }
    const long long pos = static_cast<long long>(len) + (row - first);
    const long long lp = pos / page_size;
    if (lp >= max_pages) { report(status, ROLLART_ERR_BOUNDS, static_cast<int>(lp), 1); return; }
    const int pg = __ldg(page_table + static_cast<long long>(t) * max_pages + lp);
    if (pg < 0 || pg >= num_pages) { report(status, ROLLART_ERR_BOUNDS, pg, 1); return; }
    const int slot = static_cast<int>(pos - lp * page_size);

    const long long dst = ((static_cast<long long>(pg) * num_kv_heads + h) * page_size + slot) * kVec + c;
    if constexpr (kMode == kQuantize) {
        reinterpret_cast<uint2 *>(k_pool)[dst] = quantize8(kv, k_inv_scale);
        reinterpret_cast<uint2 *>(v_pool)[dst] = quantize8(vv, v_inv_scale);
    } else {
        reinterpret_cast<uint4 *>(k_pool)[dst] = kv;
        reinterpret_cast<uint4 *>(v_pool)[dst] = vv;
    }
}

// Gather: thread -> (output row, kv head, 16-byte piece); row r of item i is the token at logical position r.
// kVec = 16-byte pieces of a row: 16 for bf16 pools, 8 for pools of 8-bit codes.
template <int kVec>
__global__ void __launch_bounds__(kThreads)
kv_gather_kernel(const void *__restrict__ k_pool, const void *__restrict__ v_pool, int num_pages,
                 int page_size, int num_kv_heads, const int32_t *__restrict__ page_table, int max_pages,
                 const int32_t *__restrict__ seq_lens, int num_traj, const int32_t *__restrict__ traj_ids,
                 const int32_t *__restrict__ out_indptr, int n_items, int total_rows, uint4 *__restrict__ k_out,
                 uint4 *__restrict__ v_out, DeviceStatus *status) {
    const long long gid = static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x;
    const long long n_vec = static_cast<long long>(total_rows) * num_kv_heads * kVec;
    if (gid >= n_vec) return;
    const int c = static_cast<int>(gid % kVec);
    const long long rh = gid / kVec;
    const int h = static_cast<int>(rh % num_kv_heads);
    const int row = static_cast<int>(rh / num_kv_heads);
    const int i = find_item(out_indptr, n_items, row);
    const int t = traj_ids ? __ldg(traj_ids + i) : i;
    if (t < 0 || t >= num_traj) { report(status, ROLLART_ERR_BOUNDS, t, 5); return; }
    const int first = __ldg(out_indptr + i);
    if (row < first || row >= __ldg(out_indptr + i + 1)) { report(status, ROLLART_ERR_BOUNDS, row, 5); return; }   // malformed out_indptr
    const int pos = row - first;
    if (pos >= __ldg(seq_lens + t)) { report(status, ROLLART_ERR_BOUNDS, pos, 5); return; }
    const int lp = pos / page_size;
    if (lp >= max_pages) { report(status, ROLLART_ERR_BOUNDS, lp, 5); return; }
    const int pg = __ldg(page_table + static_cast<long long>(t) * max_pages + lp);
    if (pg < 0 || pg >= num_pages) { report(status, ROLLART_ERR_BOUNDS, pg, 5); return; }
    const long long src = ((static_cast<long long>(pg) * num_kv_heads + h) * page_size + (pos - lp * page_size)) * kVec + c;
    k_out[gid] = __ldg(reinterpret_cast<const uint4 *>(k_pool) + src);
    v_out[gid] = __ldg(reinterpret_cast<const uint4 *>(v_pool) + src);
}

}  // namespace

cudaError_t launch_kv_gather(const rollart_kv_pool &pool, const rollart_trajs &trajs, const int32_t *traj_ids,
                             const int32_t *out_indptr, int n_items, int total_rows, void *k_out, void *v_out,
                             DeviceStatus *status, cudaStream_t stream, int64_t *launches, bool fp8) {
    const int vec = fp8 ? kVecPerRow / 2 : kVecPerRow;
    const long long n_vec = static_cast<long long>(total_rows) * pool.num_kv_heads * vec;
    if (n_vec == 0) return cudaSuccess;
    const long long blocks = (n_vec + kThreads - 1) / kThreads;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
    auto kernel = fp8 ? kv_gather_kernel<kVecPerRow / 2> : kv_gather_kernel<kVecPerRow>;
    kernel<<<static_cast<unsigned>(blocks), kThreads, 0, stream>>>(
        pool.k_pool, pool.v_pool, pool.num_pages, pool.page_size, pool.num_kv_heads, trajs.page_table,
        trajs.max_pages_per_traj, trajs.seq_lens, trajs.num_traj, traj_ids, out_indptr, n_items, total_rows,
        static_cast<uint4 *>(k_out), static_cast<uint4 *>(v_out), status);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_kv_append(const rollart_kv_pool &pool, const rollart_trajs &trajs, const int32_t *traj_ids,
                             const int32_t *new_indptr, int n_items, int total_new, const void *k_new,
                             const void *v_new, int32_t *seq_lens_out, DeviceStatus *status, cudaStream_t stream,
                             int64_t *launches, bool fp8, float k_scale, float v_scale, bool rows_are_codes) {
    const int vec = fp8 && rows_are_codes ? kVecPerRow / 2 : kVecPerRow;
    const long long n_vec = static_cast<long long>(total_new) * pool.num_kv_heads * vec;
    const long long n_thr = n_vec > n_items ? n_vec : n_items;
    if (n_thr == 0) return cudaSuccess;
    const long long blocks = (n_thr + kThreads - 1) / kThreads;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
    auto kernel = !fp8 ? kv_append_kernel<kCopyBf16> : rows_are_codes ? kv_append_kernel<kCopyCodes> : kv_append_kernel<kQuantize>;
    const bool quant = fp8 && !rows_are_codes;
    kernel<<<static_cast<unsigned>(blocks), kThreads, 0, stream>>>(
        pool.k_pool, pool.v_pool, quant ? 1.f / k_scale : 1.f, quant ? 1.f / v_scale : 1.f, pool.num_pages,
        pool.page_size, pool.num_kv_heads, trajs.page_table, trajs.max_pages_per_traj, trajs.seq_lens, trajs.num_traj,
        traj_ids, new_indptr, n_items, total_new, static_cast<const uint4 *>(k_new), static_cast<const uint4 *>(v_new),
        seq_lens_out, status);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace rollart
