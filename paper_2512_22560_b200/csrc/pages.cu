// Page bookkeeping between engine steps: reserve (a trajectory is added or grows) and release (a
// trajectory is aborted or evicted).  The free pages form a stack in device memory.  Both calls are
// all-or-nothing and deterministic: items take or return their pages in item order, with the
// positions computed by a block-wide scan, never by racing atomics.  One thread block per call: this
// is control-path work on a few thousand integers.
#include "rollart_internal.cuh"

namespace rollart {

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;

struct PageArgs {
    int32_t *free_pages;
    int32_t *free_count;
    int capacity;              // entries free_pages can hold (release only)
    int page_size;
    int32_t *page_table;
    int max_pages;
    int32_t *seq_lens;         // read by reserve, zeroed by release
    int num_traj;
    const int32_t *traj_ids;   // nullable: identity
    const int32_t *new_tokens; // reserve only
    int n_items;
    DeviceStatus *status;
};

// exclusive scan over the block's kThreads values; returns this thread's offset, *total gets the block sum
__device__ __forceinline__ int block_exclusive_scan(int v, int *warp_sums, int *total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += u;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = lane < kWarps ? warp_sums[lane] : 0;
        int wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += u;
        }
        warp_sums[lane] = wi - w;              // exclusive offset of each warp
        if (lane == 31) *total = wi;
    }
    __syncthreads();
    const int off = warp_sums[warp] + incl - v;
    __syncthreads();                           // warp_sums is reused by the next call
    return off;
}

// pages the item's trajectory has (`have`) and must have after growing (`want`); false if the item is invalid
template <bool kReserve>
__device__ __forceinline__ bool item_pages(const PageArgs &a, int i, int &t, int &have, int &want) {
    t = a.traj_ids ? __ldg(a.traj_ids + i) : i;
    if (t < 0 || t >= a.num_traj) return false;
    const int len = a.seq_lens[t];
    const int grow = kReserve ? __ldg(a.new_tokens + i) : 0;
    if (len < 0 || grow < 0) return false;
    const long long h = (static_cast<long long>(len) + a.page_size - 1) / a.page_size;
    const long long w = (static_cast<long long>(len) + grow + a.page_size - 1) / a.page_size;
    if (w > a.max_pages) return false;
    have = static_cast<int>(h);
    want = static_cast<int>(w);
    return true;
}

template <bool kReserve>
__global__ void __launch_bounds__(kThreads) pages_kernel(const PageArgs a) {
    __shared__ int s_warp[32];
    __shared__ int s_total, s_bad;
    __shared__ int s_t[kThreads], s_first[kThreads], s_count[kThreads], s_off[kThreads];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();

    // pass 1: validate everything and count the pages that move; nothing is written yet
    int mine = 0;
    for (int i = threadIdx.x; i < a.n_items; i += kThreads) {
        int t, have, want;
        if (!item_pages<kReserve>(a, i, t, have, want)) { s_bad = 1; continue; }
        mine += kReserve ? want - have : have;
    }
    int moved;
    block_exclusive_scan(mine, s_warp, &s_total);
    moved = s_total;
    const int top = *a.free_count;
    const bool fits = kReserve ? moved <= top : static_cast<long long>(top) + moved <= a.capacity;
    if (s_bad || !fits || top < 0) {
        if (threadIdx.x == 0) report(a.status, ROLLART_ERR_BOUNDS, s_bad ? -1 : moved, 6);
        return;
    }

    // pass 2: chunks of kThreads items in order; a warp moves the pages of one item
    int base = 0;
    for (int c0 = 0; c0 < a.n_items; c0 += kThreads) {
        const int i = c0 + threadIdx.x;
        int t = 0, have = 0, want = 0;
        if (i < a.n_items) item_pages<kReserve>(a, i, t, have, want);
        const int cnt = i < a.n_items ? (kReserve ? want - have : have) : 0;
        const int off = block_exclusive_scan(cnt, s_warp, &s_total);
        s_t[threadIdx.x] = t;
        s_first[threadIdx.x] = kReserve ? have : 0;
        s_count[threadIdx.x] = cnt;
        s_off[threadIdx.x] = base + off;
        __syncthreads();
        const int n_here = min(kThreads, a.n_items - c0);
        for (int it = warp; it < n_here; it += kWarps) {
            int32_t *row = a.page_table + static_cast<long long>(s_t[it]) * a.max_pages + s_first[it];
            for (int k = lane; k < s_count[it]; k += 32) {
                if (kReserve) {
                    row[k] = a.free_pages[top - 1 - (s_off[it] + k)];          // pop in item order
                } else {
                    a.free_pages[top + s_off[it] + k] = row[k];                // push in item order
                    row[k] = -1;
                }
            }
            if (!kReserve && lane == 0) a.seq_lens[s_t[it]] = 0;
        }
        base += s_total;
        __syncthreads();
    }
    if (threadIdx.x == 0) *a.free_count = kReserve ? top - moved : top + moved;
}

struct EvictArgs {
    int32_t *free_pages;
    int32_t *free_count;
    int capacity;
    int page_size;
    int32_t *page_table;
    int max_pages;
    int32_t *seq_lens;
    int num_traj;
    const int32_t *start_version;
    long long threshold;       // current version - alpha: trajectories started before it are stale
    int32_t *evicted_ids;
    int32_t *n_evicted;
    DeviceStatus *status;
};

// Stale eviction: the live trajectories whose start version lies before the window give their pages back, in
// trajectory order, exactly as the release kernel does for that list; the list itself is written out.  Selection
// and positions come from block-wide scans (a stable compaction), so the result does not depend on timing.
__global__ void __launch_bounds__(kThreads) pages_evict_kernel(const EvictArgs a) {
    __shared__ int s_warp[32];
    __shared__ int s_total, s_bad;
    __shared__ int s_count[kThreads], s_off[kThreads];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    auto stale_pages = [&](int t, bool &stale) {      // pages of trajectory t if it is stale (else 0); -1 if its length is invalid
        stale = false;
        const int len = a.seq_lens[t];
        if (len < 0) return -1;
        if (len == 0 || static_cast<long long>(__ldg(a.start_version + t)) >= a.threshold) return 0;
        const long long have = (static_cast<long long>(len) + a.page_size - 1) / a.page_size;
        if (have > a.max_pages) return -1;
        stale = true;
        return static_cast<int>(have);
    };

    // pass 1: validate and count; nothing is written yet
    int my_pages = 0, my_items = 0;
    for (int t = threadIdx.x; t < a.num_traj; t += kThreads) {
        bool stale;
        const int n = stale_pages(t, stale);
        if (n < 0) { s_bad = 1; continue; }
        my_pages += n;
        my_items += stale ? 1 : 0;
    }
    block_exclusive_scan(my_pages, s_warp, &s_total);
    const int moved = s_total;
    block_exclusive_scan(my_items, s_warp, &s_total);
    const int gone = s_total;
    const int top = *a.free_count;
    if (s_bad || top < 0 || static_cast<long long>(top) + moved > a.capacity) {
        if (threadIdx.x == 0) {
            report(a.status, ROLLART_ERR_BOUNDS, s_bad ? -1 : moved, 6);
            *a.n_evicted = 0;
        }
        return;
    }

    // pass 2: chunks of kThreads trajectories in order; a warp moves the pages of one trajectory
    int base_pages = 0, base_items = 0;
    for (int c0 = 0; c0 < a.num_traj; c0 += kThreads) {
        const int t = c0 + threadIdx.x;
        bool stale = false;
        const int cnt = t < a.num_traj ? max(0, stale_pages(t, stale)) : 0;
        const int off_pages = block_exclusive_scan(cnt, s_warp, &s_total);
        const int chunk_pages = s_total;
        const int off_items = block_exclusive_scan(stale ? 1 : 0, s_warp, &s_total);
        const int chunk_items = s_total;
        s_count[threadIdx.x] = stale ? cnt : -1;
        s_off[threadIdx.x] = base_pages + off_pages;
        if (stale) a.evicted_ids[base_items + off_items] = t;
        __syncthreads();
        const int n_here = min(kThreads, a.num_traj - c0);
        for (int it = warp; it < n_here; it += kWarps) {
            if (s_count[it] < 0) continue;
            int32_t *row = a.page_table + static_cast<long long>(c0 + it) * a.max_pages;
            for (int k = lane; k < s_count[it]; k += 32) {
                a.free_pages[top + s_off[it] + k] = row[k];                    // push in trajectory order
                row[k] = -1;
            }
            if (lane == 0) a.seq_lens[c0 + it] = 0;
        }
        base_pages += chunk_pages;
        base_items += chunk_items;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        *a.free_count = top + moved;
        *a.n_evicted = gone;
    }
}

}  // namespace

cudaError_t launch_pages(bool reserve, int32_t *free_pages, int32_t *free_count, int capacity, int page_size,
                         int32_t *page_table, int max_pages, int32_t *seq_lens, int num_traj, const int32_t *traj_ids,
                         const int32_t *new_tokens, int n_items, DeviceStatus *status, cudaStream_t stream, int64_t *launches) {
    PageArgs a{free_pages, free_count, capacity, page_size, page_table, max_pages, seq_lens, num_traj, traj_ids, new_tokens,
               n_items, status};
    if (reserve) pages_kernel<true><<<1, kThreads, 0, stream>>>(a);
    else pages_kernel<false><<<1, kThreads, 0, stream>>>(a);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_pages_evict(int32_t *free_pages, int32_t *free_count, int capacity, int page_size, int32_t *page_table,
                               int max_pages, int32_t *seq_lens, int num_traj, const int32_t *start_version,
                               int current_version, int alpha, int32_t *evicted_ids, int32_t *n_evicted, DeviceStatus *status,
                               cudaStream_t stream, int64_t *launches) {
    EvictArgs a{free_pages, free_count, capacity, page_size, page_table, max_pages, seq_lens, num_traj, start_version,
                static_cast<long long>(current_version) - static_cast<long long>(alpha), evicted_ids, n_evicted, status};
    pages_evict_kernel<<<1, kThreads, 0, stream>>>(a);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace rollart
