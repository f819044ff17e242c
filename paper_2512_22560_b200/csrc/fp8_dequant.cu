// Observation-chunk attention over fp8 pools, first half: the contexts of the listed trajectories are expanded from
// E4M3 codes to bf16 into a scratch pool of the same page geometry, and the chunk kernel then runs over the scratch
// pool.  Every finite E4M3 value is a bf16 value, so the expansion is exact; the pool scales are applied by the
// attention kernel (k_scale folded into the score scale, v_scale into the final normalisation).
//
// The chunk path is bound by the tensor cores (Sec. 3.1: prefill is the compute-bound phase), so one extra pass over
// the context at the HBM rate (1 byte read, 2 written per element) costs a few per cent of the attention itself.
//
// Scratch layout: two bf16 pools of `capacity_pages` pages, then a page table [n_items][pages_per_item]
// (pages_per_item = ceil(max_seq_len / page_size)), the lengths, and the first scratch page of every item.  The items'
// pages are packed one after the other in logical order (a plan kernel takes the running sum of ceil(len / page_size)
// on the device), so the pools need as many pages as the listed contexts hold, not n_items times the longest bound.
// One thread block expands one (item, logical page): all kv heads of a page are one contiguous run in both pools.
#include "rollart_internal.cuh"

namespace rollart {

namespace {

constexpr int kThreads = 256;

// two E4M3 codes (low 16 bits of `pair`) -> two bf16: e4m3 -> f16 -> f32 -> bf16, every step exact
__device__ __forceinline__ uint32_t e4m3x2_to_bf16x2(uint32_t pair) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(static_cast<uint16_t>(pair)));
    const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&h2));
    const __nv_bfloat162 b = __floats2bfloat162_rn(f.x, f.y);
    return *reinterpret_cast<const uint32_t *>(&b);
}

// four E4M3 codes -> four bf16.  A code's seven low bits, placed at bit 20 of an fp32 word, are its exponent and mantissa
// fields with the fp32 bias in place of the E4M3 one (a subnormal code becomes an fp32 subnormal), so one multiplication
// by 2^(127-7) gives the code's value exactly; its upper half is the bf16.  NaN codes (S.1111.111) are not covered by
// that and take the conversion instructions.
__device__ __forceinline__ void expand4(uint32_t w, uint32_t &lo, uint32_t &hi) {
    if ((((w & 0x7F7F7F7Fu) + 0x01010101u) & 0x80808080u) != 0u) {
        lo = e4m3x2_to_bf16x2(w);
        hi = e4m3x2_to_bf16x2(w >> 16);
        return;
    }
    const float up = 0x1p120f;
    const uint32_t f0 = __float_as_uint(__uint_as_float((w & 0x0000007Fu) << 20) * up);
    const uint32_t f1 = __float_as_uint(__uint_as_float((w & 0x00007F00u) << 12) * up);
    const uint32_t f2 = __float_as_uint(__uint_as_float((w & 0x007F0000u) << 4) * up);
    const uint32_t f3 = __float_as_uint(__uint_as_float((w & 0x7F000000u) >> 4) * up);
    const uint32_t sgn = w & 0x80808080u;
    lo = __byte_perm(f0, f1, 0x7632) | __byte_perm(sgn, 0u, 0x1404);      // upper halves of f0, f1; signs to bits 15 and 31
    hi = __byte_perm(f2, f3, 0x7632) | __byte_perm(sgn, 0u, 0x3424);
}

__device__ __forceinline__ void expand16(const uint4 &codes, uint4 &lo, uint4 &hi) {
    expand4(codes.x, lo.x, lo.y);
    expand4(codes.y, lo.z, lo.w);
    expand4(codes.z, hi.x, hi.y);
    expand4(codes.w, hi.z, hi.w);
}

constexpr int kPlanThreads = 1024;

// One block: validates every item, writes its length (0 for a bad item, which is reported and then attends to nothing)
// and the index of its first scratch page (running sum of the page counts, items in call order).
__global__ void __launch_bounds__(kPlanThreads)
fp8_scratch_plan_kernel(const int32_t *__restrict__ seq_lens, int num_traj, const int32_t *__restrict__ traj_ids,
                        const int32_t *__restrict__ lens_override, int n_items, int page_size, int max_pages, int max_seq_len,
                        long long capacity_pages, int32_t *__restrict__ scratch_lens, int32_t *__restrict__ first_page,
                        DeviceStatus *status) {
    __shared__ int s_warp[kPlanThreads / 32];
    __shared__ long long s_carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (int base = 0; base < n_items; base += kPlanThreads) {
        const int item = base + threadIdx.x;
        int len = 0, pages = 0;
        if (item < n_items) {
            const int t = traj_ids ? __ldg(traj_ids + item) : item;
            if (t < 0 || t >= num_traj) {
                report(status, ROLLART_ERR_BOUNDS, t, 3);
            } else {
                // lens_override (group decode): only the first lens_override[item] tokens, the group's shared prefix
                len = lens_override ? __ldg(lens_override + item) : __ldg(seq_lens + t);
                if (len < 0 || len > max_seq_len || static_cast<long long>(len) > static_cast<long long>(max_pages) * page_size) {
                    report(status, ROLLART_ERR_BOUNDS, len, 3);
                    len = 0;
                }
            }
            pages = (len + page_size - 1) / page_size;
        }
        // exclusive prefix of `pages` over the block, on top of the carry of the earlier rounds
        int incl = pages;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int w = s_warp[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o) w += v;
            }
            s_warp[lane] = w;                      // inclusive over the warps
        }
        __syncthreads();
        const long long before = s_carry + (warp > 0 ? s_warp[warp - 1] : 0) + (incl - pages);
        if (item < n_items) {
            if (before + pages > capacity_pages) {        // the scratch pools are smaller than the contexts listed
                report(status, ROLLART_ERR_WORKSPACE, item, 3);
                len = 0;
            }
            scratch_lens[item] = len;
            first_page[item] = static_cast<int32_t>(before < 0x7FFFFFFFLL ? before : 0x7FFFFFFFLL);
        }
        __syncthreads();
        if (threadIdx.x == kPlanThreads - 1) s_carry += s_warp[kPlanThreads / 32 - 1];
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kThreads)
fp8_pages_to_bf16_kernel(const uint4 *__restrict__ k_pool, const uint4 *__restrict__ v_pool, int num_pages, int page_size,
                         int num_kv_heads, const int32_t *__restrict__ page_table, int max_pages, int num_traj,
                         const int32_t *__restrict__ traj_ids, int n_items, int pages_per_item,
                         const int32_t *__restrict__ scratch_lens, const int32_t *__restrict__ first_page,
                         uint4 *__restrict__ k_scratch, uint4 *__restrict__ v_scratch, int32_t *__restrict__ scratch_table,
                         DeviceStatus *status) {
    const int item = blockIdx.x / pages_per_item;
    const int lp = blockIdx.x - item * pages_per_item;
    if (item >= n_items) return;
    const int len = __ldg(scratch_lens + item);                      // validated by the plan kernel, 0 for a bad item
    if (static_cast<long long>(lp) * page_size >= len) return;
    const int t = traj_ids ? __ldg(traj_ids + item) : item;          // in range: len > 0
    if (t < 0 || t >= num_traj) return;
    const long long s = static_cast<long long>(__ldg(first_page + item)) + lp;      // this block's scratch page
    if (threadIdx.x == 0) scratch_table[static_cast<long long>(item) * pages_per_item + lp] = static_cast<int32_t>(s);
    const int pg = __ldg(page_table + static_cast<long long>(t) * max_pages + lp);
    if (pg < 0 || pg >= num_pages) {
        if (threadIdx.x == 0) report(status, ROLLART_ERR_BOUNDS, pg, 3);
        return;
    }
    const int vec_per_page = num_kv_heads * page_size * (kHeadDim / 16);         // 16 codes per uint4
    const uint4 *ks = k_pool + static_cast<long long>(pg) * vec_per_page;
    const uint4 *vs = v_pool + static_cast<long long>(pg) * vec_per_page;
    uint4 *kd = k_scratch + s * vec_per_page * 2;
    uint4 *vd = v_scratch + s * vec_per_page * 2;
    // two pieces of K and of V per thread and round: four independent loads in flight
    for (int j = threadIdx.x; j < vec_per_page; j += 2 * kThreads) {
        const int j2 = j + kThreads;
        const bool two = j2 < vec_per_page;
        const uint4 kc = __ldg(ks + j), vc = __ldg(vs + j);
        uint4 kc2 = make_uint4(0u, 0u, 0u, 0u), vc2 = kc2;
        if (two) { kc2 = __ldg(ks + j2); vc2 = __ldg(vs + j2); }
        uint4 a, b;
        expand16(kc, a, b);
        kd[2 * j] = a;
        kd[2 * j + 1] = b;
        expand16(vc, a, b);
        vd[2 * j] = a;
        vd[2 * j + 1] = b;
        if (two) {
            expand16(kc2, a, b);
            kd[2 * j2] = a;
            kd[2 * j2 + 1] = b;
            expand16(vc2, a, b);
            vd[2 * j2] = a;
            vd[2 * j2 + 1] = b;
        }
    }
}

size_t align_up(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

}  // namespace

namespace {
// the small arrays behind the pools: page table, lengths, first page of every item
size_t tail_bytes(int n_items, int pages_per_item) {
    return align_up(static_cast<size_t>(n_items) * pages_per_item * sizeof(int32_t)) +
           2 * align_up(static_cast<size_t>(n_items) * sizeof(int32_t));
}
}  // namespace

size_t fp8_chunk_scratch_bytes(int n_items, int num_kv_heads, int page_size, int max_seq_len, long long total_pages) {
    int ppi = (max_seq_len + page_size - 1) / page_size;
    if (ppi < 1) ppi = 1;
    const long long worst = static_cast<long long>(n_items) * ppi;
    if (total_pages < 0 || total_pages > worst) total_pages = worst;
    if (total_pages < 1) total_pages = 1;
    const size_t pool_bytes = align_up(static_cast<size_t>(total_pages) * num_kv_heads * page_size * kRowBytes);
    return 2 * pool_bytes + tail_bytes(n_items, ppi);
}

Fp8ChunkScratch fp8_chunk_scratch_layout(int n_items, int num_kv_heads, int page_size, int max_seq_len, size_t scratch_bytes) {
    Fp8ChunkScratch L{};
    L.pages_per_item = (max_seq_len + page_size - 1) / page_size;
    if (L.pages_per_item < 1) L.pages_per_item = 1;
    const size_t tail = tail_bytes(n_items, L.pages_per_item);
    const size_t page_bytes = static_cast<size_t>(num_kv_heads) * page_size * kRowBytes;
    L.capacity_pages = 0;
    if (scratch_bytes > tail + 512) {
        const size_t each = ((scratch_bytes - tail) / 2) & ~static_cast<size_t>(255);     // one pool, 256-byte aligned
        L.capacity_pages = static_cast<long long>(each / page_bytes);
    }
    const long long worst = static_cast<long long>(n_items) * L.pages_per_item;
    if (L.capacity_pages > worst) L.capacity_pages = worst;
    const size_t pool_bytes = align_up(static_cast<size_t>(L.capacity_pages) * page_bytes);
    L.off_k = 0;
    L.off_v = pool_bytes;
    L.off_table = 2 * pool_bytes;
    L.off_lens = L.off_table + align_up(static_cast<size_t>(n_items) * L.pages_per_item * sizeof(int32_t));
    L.off_first = L.off_lens + align_up(static_cast<size_t>(n_items) * sizeof(int32_t));
    L.bytes = L.off_first + align_up(static_cast<size_t>(n_items) * sizeof(int32_t));
    return L;
}

cudaError_t launch_fp8_pages_to_bf16(const rollart_kv_pool &pool, const rollart_trajs &trajs, const int32_t *traj_ids,
                                     const int32_t *lens_override, int n_items, int max_seq_len, const Fp8ChunkScratch &L,
                                     void *scratch, DeviceStatus *status, cudaStream_t stream, int64_t *launches) {
    const long long blocks = static_cast<long long>(n_items) * L.pages_per_item;
    if (blocks > 0x7FFFFFFFLL || L.capacity_pages > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
    char *base = static_cast<char *>(scratch);
    int32_t *lens = reinterpret_cast<int32_t *>(base + L.off_lens), *first = reinterpret_cast<int32_t *>(base + L.off_first);
    fp8_scratch_plan_kernel<<<1, kPlanThreads, 0, stream>>>(trajs.seq_lens, trajs.num_traj, traj_ids, lens_override, n_items,
                                                            pool.page_size, trajs.max_pages_per_traj, max_seq_len,
                                                            L.capacity_pages, lens, first, status);
    ++*launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    fp8_pages_to_bf16_kernel<<<static_cast<unsigned>(blocks), kThreads, 0, stream>>>(
        static_cast<const uint4 *>(pool.k_pool), static_cast<const uint4 *>(pool.v_pool), pool.num_pages, pool.page_size,
        pool.num_kv_heads, trajs.page_table, trajs.max_pages_per_traj, trajs.num_traj, traj_ids, n_items, L.pages_per_item, lens,
        first, reinterpret_cast<uint4 *>(base + L.off_k), reinterpret_cast<uint4 *>(base + L.off_v),
        reinterpret_cast<int32_t *>(base + L.off_table), status);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace rollart
