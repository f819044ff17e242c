// Row-at-a-time attention on CUDA cores: one thread block per (query row, kv head).
//
// This is the plain path: every query row streams its keys itself, all g query heads of the
// group sharing each K/V read, with fp32 FMA dot products and warp-shuffle reductions.  It serves
// observation chunks (one block per chunk token and kv head).
#include "rollart_internal.cuh"

namespace rollart {

namespace {

constexpr int kThreads = 128;
constexpr int kWarps = kThreads / 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ int find_item(const int32_t *__restrict__ indptr, int n_items, int row) {
    int lo = 0, hi = n_items;
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (__ldg(indptr + mid) <= row) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

template <int G>
__global__ void __launch_bounds__(kThreads)
attn_rows_kernel(PoolView pool, TrajView trajs, const int32_t *__restrict__ traj_ids, const int32_t *__restrict__ q_indptr,
                 int n_items, int max_seq_len, const __nv_bfloat16 *__restrict__ q, int num_q_heads, float scale_log2,
                 __nv_bfloat16 *__restrict__ out, float *__restrict__ lse, DeviceStatus *status, int where) {
    __shared__ float sm_acc[kWarps][G][kHeadDim];
    __shared__ float sm_m[kWarps][G], sm_l[kWarps][G];

    const int row = blockIdx.x, h = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    int item = row, n_rows = 1, j_in_chunk = 0;
    if (q_indptr != nullptr) {
        item = find_item(q_indptr, n_items, row);
        const int a = __ldg(q_indptr + item);
        n_rows = __ldg(q_indptr + item + 1) - a;
        j_in_chunk = row - a;
    }
    const int t = traj_ids ? __ldg(traj_ids + item) : item;
    int count = 0;  // visible keys
    bool bad = false;
    if (t < 0 || t >= trajs.num_traj) {
        bad = true;
        if (threadIdx.x == 0) report(status, ROLLART_ERR_BOUNDS, t, where);
    } else {
        const int L = __ldg(trajs.seq_lens + t);
        if (L < 0 || L > max_seq_len || (q_indptr != nullptr && n_rows > L)) {
            bad = true;
            if (threadIdx.x == 0) report(status, ROLLART_ERR_BOUNDS, L, where);
        } else {
            count = L - n_rows + j_in_chunk + 1;
            if (L == 0) count = 0;
        }
    }
    const int begin = 0;
    const int end = bad ? 0 : count;

    // q: lane owns dims 4*lane .. 4*lane+3 of every head of the group
    float qf[G][4];
    const __nv_bfloat16 *qrow = q + (static_cast<long long>(row) * num_q_heads + h * G) * kHeadDim + lane * 4;
#pragma unroll
    for (int r = 0; r < G; ++r) {
        const uint2 raw = __ldg(reinterpret_cast<const uint2 *>(qrow + r * kHeadDim));
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.x));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.y));
        qf[r][0] = a.x; qf[r][1] = a.y; qf[r][2] = b.x; qf[r][3] = b.y;
    }

    float m[G], l[G], acc[G][4];
#pragma unroll
    for (int r = 0; r < G; ++r) {
        m[r] = -INFINITY; l[r] = 0.f;
        acc[r][0] = acc[r][1] = acc[r][2] = acc[r][3] = 0.f;
    }

    const int32_t *table_row = trajs.page_table + static_cast<long long>(t) * trajs.max_pages;
    const int P = pool.page_size;
    for (int j = begin + warp; j < end; j += kWarps) {
        const int pg = __ldg(table_row + j / P);
        if (pg < 0 || pg >= pool.num_pages) {
            if (lane == 0) report(status, ROLLART_ERR_BOUNDS, pg, where);
            continue;
        }
        const long long off = ((static_cast<long long>(pg) * pool.num_kv_heads + h) * P + (j % P)) * kHeadDim + lane * 4;
        const uint2 kraw = __ldg(reinterpret_cast<const uint2 *>(pool.k + off));
        const uint2 vraw = __ldg(reinterpret_cast<const uint2 *>(pool.v + off));
        const float2 k01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&kraw.x));
        const float2 k23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&kraw.y));
        const float2 v01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&vraw.x));
        const float2 v23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&vraw.y));
#pragma unroll
        for (int r = 0; r < G; ++r) {
            float d = qf[r][0] * k01.x + qf[r][1] * k01.y + qf[r][2] * k23.x + qf[r][3] * k23.y;
            const float s = warp_sum(d) * scale_log2;
            const float m_new = fmaxf(m[r], s);
            const float corr = exp2f(m[r] - m_new);
            // softmax weight rounded to bf16 before it multiplies V, as on the tensor-core paths
            const float p = __bfloat162float(__float2bfloat16_rn(exp2f(s - m_new)));
            m[r] = m_new;
            l[r] = l[r] * corr + p;
            acc[r][0] = acc[r][0] * corr + p * v01.x;
            acc[r][1] = acc[r][1] * corr + p * v01.y;
            acc[r][2] = acc[r][2] * corr + p * v23.x;
            acc[r][3] = acc[r][3] * corr + p * v23.y;
        }
    }

#pragma unroll
    for (int r = 0; r < G; ++r) {
        *reinterpret_cast<float4 *>(&sm_acc[warp][r][lane * 4]) = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
        if (lane == 0) { sm_m[warp][r] = m[r]; sm_l[warp][r] = l[r]; }
    }
    __syncthreads();

    // thread d merges the four warps for dim d of every head, in warp order
    const int d = threadIdx.x;
#pragma unroll
    for (int r = 0; r < G; ++r) {
        float M = sm_m[0][r];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) M = fmaxf(M, sm_m[w][r]);
        float o = 0.f, lsum = 0.f;
        if (M != -INFINITY) {
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const float a = exp2f(sm_m[w][r] - M);
                o += sm_acc[w][r][d] * a;
                lsum += sm_l[w][r] * a;
            }
        }
        const long long oi = (static_cast<long long>(row) * num_q_heads + h * G + r) * kHeadDim + d;
        out[oi] = __float2bfloat16_rn(lsum > 0.f ? o / lsum : 0.f);
        if (lse != nullptr && d == 0)
            lse[static_cast<long long>(row) * num_q_heads + h * G + r] = lsum > 0.f ? (M + log2f(lsum)) * kLn2 : -INFINITY;
    }
}

template <int G>
cudaError_t launch_rows_g(const AttnCall &c, int where, cudaStream_t stream, int64_t *launches) {
    dim3 grid(c.total_q, c.pool.num_kv_heads);
    attn_rows_kernel<G><<<grid, kThreads, 0, stream>>>(c.pool, c.trajs, c.traj_ids, c.q_indptr, c.n_items, c.max_seq_len, c.q,
                                                       c.num_q_heads, c.sm_scale * kLog2e, c.out, c.lse, c.status, where);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_rows(const AttnCall &c, int where, cudaStream_t stream, int64_t *launches) {
    const int g = c.num_q_heads / c.pool.num_kv_heads;
    switch (g) {
#define ROLLART_CASE(G) case G: return launch_rows_g<G>(c, where, stream, launches);
        ROLLART_CASE(1) ROLLART_CASE(2) ROLLART_CASE(3) ROLLART_CASE(4) ROLLART_CASE(5) ROLLART_CASE(6)
        ROLLART_CASE(7) ROLLART_CASE(8) ROLLART_CASE(9) ROLLART_CASE(10) ROLLART_CASE(11) ROLLART_CASE(12)
        ROLLART_CASE(13) ROLLART_CASE(14) ROLLART_CASE(15) ROLLART_CASE(16)
#undef ROLLART_CASE
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t launch_chunk_attn(const AttnCall &c, cudaStream_t stream, int64_t *launches, bool *too_small) {
    (void)too_small;
    return launch_rows(c, 3, stream, launches);
}

}  // namespace rollart
