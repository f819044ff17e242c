// C ABI of librollart: context, argument validation, dispatch to the kernel launchers.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

#include "rollart_internal.cuh"

using namespace rollart;

struct rollart_ctx {
    int device;
    int sm_count;
    void *workspace;
    size_t workspace_bytes;
    DeviceStatus *d_status;  // followed, 256 bytes on, by the chunk calls' bitmap of units to compute again and their unit counter
    uint32_t *d_redo;
    DeviceStatus *h_status;  // pinned
    int64_t launches;
    TmaCache tma;
    char err[320];
};

namespace {

rollart_status fail(rollart_ctx *ctx, rollart_status st, const char *fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof ctx->err, fmt, ap);
        va_end(ap);
    }
    return st;
}

rollart_status cuda_fail(rollart_ctx *ctx, cudaError_t e, const char *what) {
    return fail(ctx, ROLLART_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

rollart_status check_pool(rollart_ctx *ctx, const rollart_kv_pool *pool) {
    if (!pool || !pool->k_pool || !pool->v_pool) return fail(ctx, ROLLART_ERR_INVALID_ARG, "pool or pool pointers NULL");
    if (pool->num_pages <= 0 || pool->num_kv_heads <= 0)
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "num_pages and num_kv_heads must be positive");
    if (pool->head_dim != kHeadDim) return fail(ctx, ROLLART_ERR_UNSUPPORTED, "head_dim %d (only 128)", pool->head_dim);
    if (pool->page_size != 16 && pool->page_size != 32 && pool->page_size != 64)
        return fail(ctx, ROLLART_ERR_UNSUPPORTED, "page_size %d (only 16, 32, 64)", pool->page_size);
    if (!aligned16(pool->k_pool) || !aligned16(pool->v_pool))
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "pools must be 16-byte aligned");
    return ROLLART_OK;
}

rollart_status check_trajs(rollart_ctx *ctx, const rollart_trajs *t) {
    if (!t || !t->page_table || !t->seq_lens) return fail(ctx, ROLLART_ERR_INVALID_ARG, "trajs or its pointers NULL");
    if (t->num_traj <= 0 || t->max_pages_per_traj <= 0)
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "num_traj and max_pages_per_traj must be positive");
    return ROLLART_OK;
}

rollart_status check_heads(rollart_ctx *ctx, const rollart_kv_pool *pool, int num_q_heads) {
    if (num_q_heads <= 0 || num_q_heads % pool->num_kv_heads != 0)
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "num_q_heads %d is not a positive multiple of num_kv_heads %d",
                    num_q_heads, pool->num_kv_heads);
    if (num_q_heads / pool->num_kv_heads > kMaxGroup)
        return fail(ctx, ROLLART_ERR_UNSUPPORTED, "%d query heads per kv head (at most %d)",
                    num_q_heads / pool->num_kv_heads, kMaxGroup);
    return ROLLART_OK;
}

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

AttnCall make_call(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs, const int32_t *traj_ids,
                   const int32_t *q_indptr, int n_items, int total_q, int max_seq_len, const void *q, int num_q_heads,
                   float sm_scale, void *out, float *lse) {
    AttnCall c;
    c.pool = PoolView{static_cast<const __nv_bfloat16 *>(pool->k_pool), static_cast<const __nv_bfloat16 *>(pool->v_pool),
                      pool->num_pages, pool->page_size, pool->num_kv_heads};
    c.trajs = TrajView{trajs->page_table, trajs->seq_lens, trajs->max_pages_per_traj, trajs->num_traj};
    c.traj_ids = traj_ids;
    c.q_indptr = q_indptr;
    c.n_items = n_items;
    c.total_q = total_q;
    c.max_seq_len = max_seq_len;
    c.q = static_cast<const __nv_bfloat16 *>(q);
    c.num_q_heads = num_q_heads;
    c.sm_scale = sm_scale;
    c.out = static_cast<__nv_bfloat16 *>(out);
    c.lse = lse;
    c.workspace = ctx->workspace;
    c.workspace_bytes = ctx->workspace_bytes;
    c.status = ctx->d_status;
    c.sm_count = ctx->sm_count;
    c.tma = &ctx->tma;
    c.k_new = nullptr;
    c.v_new = nullptr;
    c.seq_lens_out = nullptr;
    c.page_offset = nullptr;
    c.shared_lens = nullptr;
    c.out_f32 = nullptr;
    c.item_order = nullptr;
    c.redo_bits = ctx->d_redo;
    c.fp8 = false;
    c.k_scale = 1.f;
    c.v_scale = 1.f;
    return c;
}

}  // namespace

extern "C" {

size_t rollart_workspace_size(int32_t max_items, int32_t num_q_heads, int32_t num_kv_heads, int32_t max_seq_len) {
    if (max_items <= 0 || num_q_heads <= 0 || num_kv_heads <= 0 || max_seq_len < 0) return 0;
    return decode_workspace_bytes(max_items, num_q_heads, num_kv_heads, max_seq_len, /*sm_count=*/0);
}

rollart_status rollart_create(rollart_ctx **out, int device, size_t workspace_bytes) {
    if (!out) return ROLLART_ERR_INVALID_ARG;
    *out = nullptr;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) return ROLLART_ERR_CUDA;
    DeviceGuard guard(device);
    if (!guard.ok) return ROLLART_ERR_CUDA;
    rollart_ctx *ctx = new (std::nothrow) rollart_ctx();
    if (!ctx) return ROLLART_ERR_CUDA;
    std::memset(ctx, 0, sizeof *ctx);
    ctx->device = device;
    cudaDeviceProp prop;
    cudaError_t e = cudaGetDeviceProperties(&prop, device);
    if (e == cudaSuccess && prop.major != 10) {
        // the kernels are sm_100a binaries; refuse loudly rather than fail at the first launch
        delete ctx;
        return ROLLART_ERR_UNSUPPORTED;
    }
    if (e == cudaSuccess) ctx->sm_count = prop.multiProcessorCount;
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_status, 256 + kChunkRedoBits / 8 + 64);
    if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, 256 + kChunkRedoBits / 8 + 64);
    if (e == cudaSuccess) ctx->d_redo = reinterpret_cast<uint32_t *>(reinterpret_cast<char *>(ctx->d_status) + 256);
    if (e == cudaSuccess) e = cudaMallocHost(&ctx->h_status, sizeof(DeviceStatus));
    if (e == cudaSuccess && workspace_bytes) e = cudaMalloc(&ctx->workspace, workspace_bytes);
    if (e == cudaSuccess && workspace_bytes) e = cudaMemset(ctx->workspace, 0, workspace_bytes);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        cudaGetLastError();
        if (ctx->workspace) cudaFree(ctx->workspace);
        if (ctx->d_status) cudaFree(ctx->d_status);
        if (ctx->h_status) cudaFreeHost(ctx->h_status);
        delete ctx;
        return ROLLART_ERR_CUDA;
    }
    ctx->workspace_bytes = workspace_bytes;
    std::snprintf(ctx->err, sizeof ctx->err, "ok");
    *out = ctx;
    return ROLLART_OK;
}

rollart_status rollart_destroy(rollart_ctx *ctx) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaDeviceSynchronize();
    if (ctx->workspace) cudaFree(ctx->workspace);
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->h_status) cudaFreeHost(ctx->h_status);
    delete ctx;
    return ROLLART_OK;
}

namespace {
rollart_status append_impl(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                           const int32_t *traj_ids, const int32_t *new_indptr, int32_t n_items, int32_t total_new,
                           const void *k_new, const void *v_new, int32_t *seq_lens_out, void *stream, bool fp8,
                           float k_scale, float v_scale, bool rows_are_codes = false) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    rollart_status st;
    if ((st = check_pool(ctx, pool)) != ROLLART_OK) return st;
    if ((st = check_trajs(ctx, trajs)) != ROLLART_OK) return st;
    if (n_items < 0 || total_new < 0) return fail(ctx, ROLLART_ERR_INVALID_ARG, "negative n_items or total_new");
    if (n_items == 0) return ROLLART_OK;
    if (!new_indptr) return fail(ctx, ROLLART_ERR_INVALID_ARG, "new_indptr NULL");
    if (total_new > 0 && (!k_new || !v_new)) return fail(ctx, ROLLART_ERR_INVALID_ARG, "k_new or v_new NULL");
    if (!aligned16(k_new) || !aligned16(v_new)) return fail(ctx, ROLLART_ERR_INVALID_ARG, "k_new/v_new must be 16-byte aligned");
    if (seq_lens_out) {
        const char *a = reinterpret_cast<const char *>(trajs->seq_lens);
        const char *b = reinterpret_cast<const char *>(seq_lens_out);
        size_t bytes = sizeof(int32_t) * static_cast<size_t>(trajs->num_traj);
        if (a < b + bytes && b < a + bytes) return fail(ctx, ROLLART_ERR_INVALID_ARG, "seq_lens_out overlaps seq_lens");
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, ROLLART_ERR_CUDA, "cannot select device %d", ctx->device);
    cudaError_t e = launch_kv_append(*pool, *trajs, traj_ids, new_indptr, n_items, total_new, k_new, v_new, seq_lens_out,
                                     ctx->d_status, static_cast<cudaStream_t>(stream), &ctx->launches, fp8, k_scale, v_scale,
                                     rows_are_codes);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "kv_append launch");
    return ROLLART_OK;
}
}  // namespace

rollart_status rollart_kv_append(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                 const int32_t *traj_ids, const int32_t *new_indptr, int32_t n_items,
                                 int32_t total_new, const void *k_new, const void *v_new, int32_t *seq_lens_out,
                                 void *stream) {
    return append_impl(ctx, pool, trajs, traj_ids, new_indptr, n_items, total_new, k_new, v_new, seq_lens_out, stream, false,
                       1.f, 1.f);
}

rollart_status rollart_kv_append_fp8(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                     const int32_t *traj_ids, const int32_t *new_indptr, int32_t n_items,
                                     int32_t total_new, const void *k_new, const void *v_new, float k_scale, float v_scale,
                                     int32_t *seq_lens_out, void *stream) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    if (!(k_scale > 0.f) || !(v_scale > 0.f) || !isfinite(k_scale) || !isfinite(v_scale))
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "k_scale and v_scale must be positive and finite");
    return append_impl(ctx, pool, trajs, traj_ids, new_indptr, n_items, total_new, k_new, v_new, seq_lens_out, stream, true,
                       k_scale, v_scale);
}

rollart_status rollart_kv_append_fp8_codes(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                           const int32_t *traj_ids, const int32_t *new_indptr, int32_t n_items,
                                           int32_t total_new, const void *k_codes, const void *v_codes,
                                           int32_t *seq_lens_out, void *stream) {
    return append_impl(ctx, pool, trajs, traj_ids, new_indptr, n_items, total_new, k_codes, v_codes, seq_lens_out, stream, true,
                       1.f, 1.f, true);
}

namespace {
rollart_status gather_impl(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                           const int32_t *traj_ids, const int32_t *out_indptr, int32_t n_items, int32_t total_rows,
                           void *k_out, void *v_out, void *stream, bool fp8) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    rollart_status st;
    if ((st = check_pool(ctx, pool)) != ROLLART_OK) return st;
    if ((st = check_trajs(ctx, trajs)) != ROLLART_OK) return st;
    if (n_items < 0 || total_rows < 0) return fail(ctx, ROLLART_ERR_INVALID_ARG, "negative n_items or total_rows");
    if (n_items == 0 || total_rows == 0) return ROLLART_OK;
    if (!out_indptr || !k_out || !v_out) return fail(ctx, ROLLART_ERR_INVALID_ARG, "out_indptr, k_out or v_out NULL");
    if (!aligned16(k_out) || !aligned16(v_out)) return fail(ctx, ROLLART_ERR_INVALID_ARG, "k_out/v_out must be 16-byte aligned");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, ROLLART_ERR_CUDA, "cannot select device %d", ctx->device);
    cudaError_t e = launch_kv_gather(*pool, *trajs, traj_ids, out_indptr, n_items, total_rows, k_out, v_out, ctx->d_status,
                                     static_cast<cudaStream_t>(stream), &ctx->launches, fp8);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "kv_gather launch");
    return ROLLART_OK;
}
}  // namespace

rollart_status rollart_kv_gather(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                 const int32_t *traj_ids, const int32_t *out_indptr, int32_t n_items, int32_t total_rows,
                                 void *k_out, void *v_out, void *stream) {
    return gather_impl(ctx, pool, trajs, traj_ids, out_indptr, n_items, total_rows, k_out, v_out, stream, false);
}

rollart_status rollart_kv_gather_fp8(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                     const int32_t *traj_ids, const int32_t *out_indptr, int32_t n_items, int32_t total_rows,
                                     void *k_out, void *v_out, void *stream) {
    return gather_impl(ctx, pool, trajs, traj_ids, out_indptr, n_items, total_rows, k_out, v_out, stream, true);
}

static rollart_status pages_common(rollart_ctx *ctx, bool reserve, int32_t *free_pages, int32_t *free_count, int32_t capacity,
                                   int32_t page_size, int32_t *page_table, int32_t max_pages, int32_t *seq_lens,
                                   int32_t num_traj, const int32_t *traj_ids, const int32_t *new_tokens, int32_t n_items,
                                   void *stream) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    if (!free_pages || !free_count || !page_table || !seq_lens) return fail(ctx, ROLLART_ERR_INVALID_ARG, "NULL pointer");
    if (page_size <= 0 || max_pages <= 0 || num_traj <= 0 || n_items < 0 || capacity < 0)
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "sizes must be positive");
    if (n_items == 0) return ROLLART_OK;
    if (reserve && !new_tokens) return fail(ctx, ROLLART_ERR_INVALID_ARG, "new_tokens NULL");
    if (!reserve && !traj_ids) return fail(ctx, ROLLART_ERR_INVALID_ARG, "traj_ids NULL");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, ROLLART_ERR_CUDA, "cannot select device %d", ctx->device);
    cudaError_t e = launch_pages(reserve, free_pages, free_count, capacity, page_size, page_table, max_pages, seq_lens, num_traj,
                                 traj_ids, new_tokens, n_items, ctx->d_status, static_cast<cudaStream_t>(stream), &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, reserve ? "pages_reserve launch" : "pages_release launch");
    return ROLLART_OK;
}

rollart_status rollart_pages_reserve(rollart_ctx *ctx, int32_t *free_pages, int32_t *free_count, int32_t page_size,
                                     int32_t *page_table, int32_t max_pages_per_traj, const int32_t *seq_lens,
                                     int32_t num_traj, const int32_t *traj_ids, const int32_t *new_tokens, int32_t n_items,
                                     void *stream) {
    return pages_common(ctx, true, free_pages, free_count, 0, page_size, page_table, max_pages_per_traj,
                        const_cast<int32_t *>(seq_lens), num_traj, traj_ids, new_tokens, n_items, stream);
}

rollart_status rollart_pages_release(rollart_ctx *ctx, int32_t *free_pages, int32_t *free_count, int32_t capacity,
                                     int32_t page_size, int32_t *page_table, int32_t max_pages_per_traj, int32_t *seq_lens,
                                     int32_t num_traj, const int32_t *traj_ids, int32_t n_items, void *stream) {
    return pages_common(ctx, false, free_pages, free_count, capacity, page_size, page_table, max_pages_per_traj, seq_lens,
                        num_traj, traj_ids, nullptr, n_items, stream);
}

rollart_status rollart_pages_evict_stale(rollart_ctx *ctx, int32_t *free_pages, int32_t *free_count, int32_t capacity,
                                         int32_t page_size, int32_t *page_table, int32_t max_pages_per_traj, int32_t *seq_lens,
                                         int32_t num_traj, const int32_t *start_version, int32_t current_version, int32_t alpha,
                                         int32_t *evicted_ids, int32_t *n_evicted, void *stream) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    if (!free_pages || !free_count || !page_table || !seq_lens || !start_version || !evicted_ids || !n_evicted)
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "NULL pointer");
    if (page_size <= 0 || max_pages_per_traj <= 0 || num_traj <= 0 || capacity < 0)
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "sizes must be positive");
    if (alpha < 0) return fail(ctx, ROLLART_ERR_INVALID_ARG, "alpha must not be negative");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, ROLLART_ERR_CUDA, "cannot select device %d", ctx->device);
    cudaError_t e = launch_pages_evict(free_pages, free_count, capacity, page_size, page_table, max_pages_per_traj, seq_lens,
                                       num_traj, start_version, current_version, alpha, evicted_ids, n_evicted, ctx->d_status,
                                       static_cast<cudaStream_t>(stream), &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "pages_evict_stale launch");
    return ROLLART_OK;
}

// max_seq_len is only an upper bound: a page-table row cannot hold more than this anyway
static int32_t clamp_bound(const rollart_kv_pool *pool, const rollart_trajs *trajs, int32_t max_seq_len) {
    const int64_t cap = static_cast<int64_t>(trajs->max_pages_per_traj) * pool->page_size;
    return static_cast<int64_t>(max_seq_len) > cap ? static_cast<int32_t>(cap > 0x7FFFFFFF ? 0x7FFFFFFF : cap) : max_seq_len;
}

static rollart_status attn_common(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                  int32_t n_items, int32_t total_q, int32_t max_seq_len, const void *q,
                                  int32_t num_q_heads, void *out) {
    rollart_status st;
    if ((st = check_pool(ctx, pool)) != ROLLART_OK) return st;
    if ((st = check_trajs(ctx, trajs)) != ROLLART_OK) return st;
    if ((st = check_heads(ctx, pool, num_q_heads)) != ROLLART_OK) return st;
    if (n_items < 0 || total_q < 0 || max_seq_len < 0)
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "negative n_items, total_q or max_seq_len");
    if (total_q > 0 && (!q || !out)) return fail(ctx, ROLLART_ERR_INVALID_ARG, "q or out NULL");
    if (!aligned16(q) || !aligned16(out)) return fail(ctx, ROLLART_ERR_INVALID_ARG, "q/out must be 16-byte aligned");
    return ROLLART_OK;
}

rollart_status rollart_decode_attn(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                   const int32_t *traj_ids, int32_t n_items, int32_t max_seq_len, const void *q,
                                   int32_t num_q_heads, float sm_scale, void *out, float *lse, void *stream) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    rollart_status st = attn_common(ctx, pool, trajs, n_items, n_items, max_seq_len, q, num_q_heads, out);
    if (st != ROLLART_OK) return st;
    if (n_items == 0) return ROLLART_OK;
    max_seq_len = clamp_bound(pool, trajs, max_seq_len);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, ROLLART_ERR_CUDA, "cannot select device %d", ctx->device);
    AttnCall c = make_call(ctx, pool, trajs, traj_ids, nullptr, n_items, n_items, max_seq_len, q, num_q_heads, sm_scale,
                           out, lse);
    bool too_small = false;
    cudaError_t e = launch_decode_attn(c, static_cast<cudaStream_t>(stream), &ctx->launches, &too_small);
    if (too_small)
        return fail(ctx, ROLLART_ERR_WORKSPACE, "workspace of %zu bytes is too small (need %zu)", ctx->workspace_bytes,
                    decode_workspace_bytes(n_items, num_q_heads, pool->num_kv_heads, max_seq_len, ctx->sm_count));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "decode_attn launch");
    return ROLLART_OK;
}

rollart_status rollart_decode_attn_fp8(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                       const int32_t *traj_ids, int32_t n_items, int32_t max_seq_len, const void *q,
                                       int32_t num_q_heads, float sm_scale, float k_scale, float v_scale, void *out,
                                       float *lse, void *stream) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    rollart_status st = attn_common(ctx, pool, trajs, n_items, n_items, max_seq_len, q, num_q_heads, out);
    if (st != ROLLART_OK) return st;
    if (!(k_scale > 0.f) || !(v_scale > 0.f) || !isfinite(k_scale) || !isfinite(v_scale))
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "k_scale and v_scale must be positive and finite");
    if (n_items == 0) return ROLLART_OK;
    max_seq_len = clamp_bound(pool, trajs, max_seq_len);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, ROLLART_ERR_CUDA, "cannot select device %d", ctx->device);
    AttnCall c = make_call(ctx, pool, trajs, traj_ids, nullptr, n_items, n_items, max_seq_len, q, num_q_heads, sm_scale,
                           out, lse);
    c.fp8 = true;
    c.k_scale = k_scale;
    c.v_scale = v_scale;
    bool too_small = false;
    cudaError_t e = launch_decode_attn(c, static_cast<cudaStream_t>(stream), &ctx->launches, &too_small);
    if (too_small)
        return fail(ctx, ROLLART_ERR_WORKSPACE, "workspace of %zu bytes is too small (need %zu)", ctx->workspace_bytes,
                    decode_workspace_bytes(n_items, num_q_heads, pool->num_kv_heads, max_seq_len, ctx->sm_count));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "decode_attn_fp8 launch");
    return ROLLART_OK;
}

namespace {
rollart_status append_decode_impl(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                  const int32_t *traj_ids, int32_t n_items, int32_t max_seq_len, const void *k_new,
                                  const void *v_new, const void *q, int32_t num_q_heads, float sm_scale, void *out,
                                  float *lse, int32_t *seq_lens_out, void *stream, bool fp8, float k_scale, float v_scale) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    rollart_status st = attn_common(ctx, pool, trajs, n_items, n_items, max_seq_len, q, num_q_heads, out);
    if (st != ROLLART_OK) return st;
    if (n_items == 0) return ROLLART_OK;
    if (!k_new || !v_new) return fail(ctx, ROLLART_ERR_INVALID_ARG, "k_new or v_new NULL");
    if (!aligned16(k_new) || !aligned16(v_new)) return fail(ctx, ROLLART_ERR_INVALID_ARG, "k_new/v_new must be 16-byte aligned");
    if (seq_lens_out) {
        const char *a = reinterpret_cast<const char *>(trajs->seq_lens);
        const char *b = reinterpret_cast<const char *>(seq_lens_out);
        size_t bytes = sizeof(int32_t) * static_cast<size_t>(trajs->num_traj);
        if (a < b + bytes && b < a + bytes) return fail(ctx, ROLLART_ERR_INVALID_ARG, "seq_lens_out overlaps seq_lens");
    }
    max_seq_len = clamp_bound(pool, trajs, max_seq_len);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, ROLLART_ERR_CUDA, "cannot select device %d", ctx->device);
    AttnCall c = make_call(ctx, pool, trajs, traj_ids, nullptr, n_items, n_items, max_seq_len, q, num_q_heads, sm_scale,
                           out, lse);
    c.k_new = static_cast<const __nv_bfloat16 *>(k_new);
    c.v_new = static_cast<const __nv_bfloat16 *>(v_new);
    c.seq_lens_out = seq_lens_out;
    c.fp8 = fp8;
    c.k_scale = k_scale;
    c.v_scale = v_scale;
    bool too_small = false;
    cudaError_t e = launch_decode_attn(c, static_cast<cudaStream_t>(stream), &ctx->launches, &too_small);
    if (too_small)
        return fail(ctx, ROLLART_ERR_WORKSPACE, "workspace of %zu bytes is too small (need %zu)", ctx->workspace_bytes,
                    decode_workspace_bytes(n_items, num_q_heads, pool->num_kv_heads, max_seq_len, ctx->sm_count));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "append_decode_attn launch");
    return ROLLART_OK;
}
}  // namespace

rollart_status rollart_append_decode_attn(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                          const int32_t *traj_ids, int32_t n_items, int32_t max_seq_len, const void *k_new,
                                          const void *v_new, const void *q, int32_t num_q_heads, float sm_scale, void *out,
                                          float *lse, int32_t *seq_lens_out, void *stream) {
    return append_decode_impl(ctx, pool, trajs, traj_ids, n_items, max_seq_len, k_new, v_new, q, num_q_heads, sm_scale, out,
                              lse, seq_lens_out, stream, false, 1.f, 1.f);
}

size_t rollart_host_staging_size(int32_t n_items, int32_t num_q_heads, int32_t num_kv_heads) {
    if (n_items <= 0 || num_q_heads <= 0 || num_kv_heads <= 0) return 0;
    return (static_cast<size_t>(n_items) * num_q_heads + 2 * static_cast<size_t>(n_items) * num_kv_heads) * kRowBytes;
}

rollart_status rollart_append_decode_attn_host(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                               const int32_t *traj_ids, int32_t n_items, int32_t max_seq_len,
                                               const void *k_new_host, const void *v_new_host, const void *q_host,
                                               int32_t num_q_heads, float sm_scale, void *out, float *lse,
                                               int32_t *seq_lens_out, void *staging, size_t staging_bytes, void *stream) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    rollart_status st = attn_common(ctx, pool, trajs, n_items, n_items, max_seq_len, q_host, num_q_heads, out);
    if (st != ROLLART_OK) return st;
    if (n_items == 0) return ROLLART_OK;
    if (!k_new_host || !v_new_host) return fail(ctx, ROLLART_ERR_INVALID_ARG, "k_new or v_new NULL");
    if (!aligned16(k_new_host) || !aligned16(v_new_host)) return fail(ctx, ROLLART_ERR_INVALID_ARG, "k_new/v_new must be 16-byte aligned");
    const size_t need = rollart_host_staging_size(n_items, num_q_heads, pool->num_kv_heads);
    if (!staging || (reinterpret_cast<uintptr_t>(staging) & 255u) != 0)
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "staging must be a 256-byte aligned device buffer");
    if (staging_bytes < need) return fail(ctx, ROLLART_ERR_WORKSPACE, "staging of %zu bytes is too small (need %zu)", staging_bytes, need);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, ROLLART_ERR_CUDA, "cannot select device %d", ctx->device);
    // what the step itself would refuse is refused before the copy is enqueued
    if (seq_lens_out) {
        const char *a = reinterpret_cast<const char *>(trajs->seq_lens);
        const char *b = reinterpret_cast<const char *>(seq_lens_out);
        size_t bytes = sizeof(int32_t) * static_cast<size_t>(trajs->num_traj);
        if (a < b + bytes && b < a + bytes) return fail(ctx, ROLLART_ERR_INVALID_ARG, "seq_lens_out overlaps seq_lens");
    }
    {
        const size_t ws = decode_workspace_bytes(n_items, num_q_heads, pool->num_kv_heads, clamp_bound(pool, trajs, max_seq_len),
                                                 ctx->sm_count);
        if (!ctx->workspace || ws > ctx->workspace_bytes)
            return fail(ctx, ROLLART_ERR_WORKSPACE, "workspace of %zu bytes is too small (need %zu)", ctx->workspace_bytes, ws);
    }
    const size_t q_bytes = static_cast<size_t>(n_items) * num_q_heads * kRowBytes;        // multiples of 256
    const size_t kv_bytes = static_cast<size_t>(n_items) * pool->num_kv_heads * kRowBytes;
    char *sb = static_cast<char *>(staging);
    void *sq = sb, *sk = sb + q_bytes, *sv = sb + q_bytes + kv_bytes;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const char *hq = static_cast<const char *>(q_host);
    cudaError_t e = cudaErrorInvalidValue;
    if (hq + q_bytes == k_new_host && hq + q_bytes + kv_bytes == v_new_host) {
        // the three buffers follow one another in host memory (q, k_new, v_new): one copy moves them all, provided
        // they are parts of one page-locked allocation (a copy across two allocations is refused up front)
        e = cudaMemcpyAsync(sq, q_host, q_bytes + 2 * kv_bytes, cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) cudaGetLastError();
    }
    if (e != cudaSuccess) {
        e = cudaMemcpyAsync(sq, q_host, q_bytes, cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess) e = cudaMemcpyAsync(sk, k_new_host, kv_bytes, cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess) e = cudaMemcpyAsync(sv, v_new_host, kv_bytes, cudaMemcpyHostToDevice, s);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e, "host -> device copy");
    return append_decode_impl(ctx, pool, trajs, traj_ids, n_items, max_seq_len, sk, sv, sq, num_q_heads, sm_scale, out, lse,
                              seq_lens_out, stream, false, 1.f, 1.f);
}

rollart_status rollart_append_decode_attn_fp8(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                              const int32_t *traj_ids, int32_t n_items, int32_t max_seq_len,
                                              const void *k_new, const void *v_new, const void *q, int32_t num_q_heads,
                                              float sm_scale, float k_scale, float v_scale, void *out, float *lse,
                                              int32_t *seq_lens_out, void *stream) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    if (!(k_scale > 0.f) || !(v_scale > 0.f) || !isfinite(k_scale) || !isfinite(v_scale))
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "k_scale and v_scale must be positive and finite");
    return append_decode_impl(ctx, pool, trajs, traj_ids, n_items, max_seq_len, k_new, v_new, q, num_q_heads, sm_scale, out,
                              lse, seq_lens_out, stream, true, k_scale, v_scale);
}

namespace {
// Workspace of a group decode call: the decode kernel's own workspace first, then these arrays.
struct GroupLayout {
    size_t group_traj, item_off, group_order, lse_a, lse_b, part_a, part_b, total;
};
GroupLayout group_layout(int n_items, int num_q_heads, int num_kv_heads, int max_seq_len, int sm_count) {
    auto up = [](size_t x) { return (x + 255) & ~size_t(255); };
    const size_t rows = static_cast<size_t>(n_items) * num_q_heads;
    GroupLayout g;
    size_t at = up(decode_workspace_bytes(n_items, num_q_heads, num_kv_heads, max_seq_len, sm_count));
    g.group_traj = at; at += up(sizeof(int32_t) * static_cast<size_t>(n_items));
    g.item_off = at;   at += up(sizeof(int32_t) * static_cast<size_t>(n_items));
    g.group_order = at; at += up(sizeof(int32_t) * static_cast<size_t>(n_items));
    g.lse_a = at;      at += up(sizeof(float) * rows);
    g.lse_b = at;      at += up(sizeof(float) * rows);
    g.part_a = at;     at += up(sizeof(float) * rows * kHeadDim);
    g.part_b = at;     at += up(sizeof(float) * rows * kHeadDim);
    g.total = at;
    return g;
}
}  // namespace

size_t rollart_group_decode_workspace_size(int32_t max_items, int32_t num_q_heads, int32_t num_kv_heads, int32_t max_seq_len) {
    if (max_items <= 0 || num_q_heads <= 0 || num_kv_heads <= 0 || max_seq_len < 0) return 0;
    return group_layout(max_items, num_q_heads, num_kv_heads, max_seq_len, /*sm_count=*/0).total;
}

static rollart_status group_decode_impl(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                        const int32_t *traj_ids, int32_t n_items, const int32_t *group_indptr,
                                        const int32_t *shared_lens, int32_t n_groups, int32_t max_seq_len, const void *q,
                                        int32_t num_q_heads, float sm_scale, void *out, float *lse, void *stream_, bool fp8,
                                        float k_scale, float v_scale, void *scratch, size_t scratch_bytes) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    rollart_status st = attn_common(ctx, pool, trajs, n_items, n_items, max_seq_len, q, num_q_heads, out);
    if (st != ROLLART_OK) return st;
    if (fp8 && (!(k_scale > 0.f) || !(v_scale > 0.f) || !isfinite(k_scale) || !isfinite(v_scale)))
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "k_scale and v_scale must be positive and finite");
    if (n_groups < 0 || n_groups > n_items) return fail(ctx, ROLLART_ERR_INVALID_ARG, "n_groups must lie in [0, n_items]");
    if (n_items == 0) return ROLLART_OK;
    if (n_groups == 0) return fail(ctx, ROLLART_ERR_INVALID_ARG, "items without groups");
    if (!group_indptr || !shared_lens) return fail(ctx, ROLLART_ERR_INVALID_ARG, "group_indptr or shared_lens NULL");
    max_seq_len = clamp_bound(pool, trajs, max_seq_len);
    const GroupLayout lay = group_layout(n_items, num_q_heads, pool->num_kv_heads, max_seq_len, ctx->sm_count);
    if (!ctx->workspace || lay.total > ctx->workspace_bytes)
        return fail(ctx, ROLLART_ERR_WORKSPACE, "workspace of %zu bytes is too small (need %zu)", ctx->workspace_bytes, lay.total);
    Fp8ChunkScratch sl{};
    if (fp8) {
        // the prefixes (one per group) are expanded to bf16 for the tensor-core kernel; the private parts are read as codes
        sl = fp8_chunk_scratch_layout(n_groups, pool->num_kv_heads, pool->page_size, max_seq_len, scratch_bytes);
        if (!scratch || (reinterpret_cast<uintptr_t>(scratch) & 255u) != 0)
            return fail(ctx, ROLLART_ERR_INVALID_ARG, "scratch must be a 256-byte aligned device buffer");
        if (sl.capacity_pages < 1)
            return fail(ctx, ROLLART_ERR_WORKSPACE, "scratch of %zu bytes cannot hold a single page", scratch_bytes);
        if (static_cast<long long>(n_groups) * sl.pages_per_item > 0x7FFFFFFFLL)
            return fail(ctx, ROLLART_ERR_UNSUPPORTED, "too many scratch pages");
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, ROLLART_ERR_CUDA, "cannot select device %d", ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    char *ws = static_cast<char *>(ctx->workspace);
    int32_t *group_traj = reinterpret_cast<int32_t *>(ws + lay.group_traj);
    int32_t *item_off = reinterpret_cast<int32_t *>(ws + lay.item_off);
    int32_t *group_order = reinterpret_cast<int32_t *>(ws + lay.group_order);
    float *lse_a = reinterpret_cast<float *>(ws + lay.lse_a), *lse_b = reinterpret_cast<float *>(ws + lay.lse_b);
    float *part_a = reinterpret_cast<float *>(ws + lay.part_a), *part_b = reinterpret_cast<float *>(ws + lay.part_b);

    // items that a broken indptr leaves out of every group still get a defined offset
    cudaError_t e = cudaMemsetAsync(ws + lay.group_traj, 0, lay.lse_a - lay.group_traj, stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "group_decode_attn memset");
    AttnCall base = make_call(ctx, pool, trajs, traj_ids, nullptr, n_items, n_items, max_seq_len, q, num_q_heads, sm_scale,
                              out, lse);
    e = launch_group_prepare(base.trajs, traj_ids, n_items, group_indptr, shared_lens, n_groups, pool->page_size, group_traj,
                             item_off, group_order, ctx->d_status, stream, &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "group_decode_attn prepare launch");

    bool too_small = false;
    // shared prefix: the members' query rows of one group form the rows of an M-tile; every row sees the whole prefix
    AttnCall sc = base;
    sc.traj_ids = group_traj;
    sc.q_indptr = group_indptr;
    sc.n_items = n_groups;
    sc.shared_lens = shared_lens;
    sc.out_f32 = part_a;
    sc.lse = lse_a;
    sc.item_order = group_order;        // longest prefixes first: the blocks of this pass differ a lot in length
    if (fp8) {
        e = launch_fp8_pages_to_bf16(*pool, *trajs, group_traj, shared_lens, n_groups, max_seq_len, sl, scratch, ctx->d_status,
                                     stream, &ctx->launches);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "group_decode_attn fp8 expansion launch");
        char *sb = static_cast<char *>(scratch);
        sc.pool = PoolView{reinterpret_cast<const __nv_bfloat16 *>(sb + sl.off_k), reinterpret_cast<const __nv_bfloat16 *>(sb + sl.off_v),
                           static_cast<int>(sl.capacity_pages), pool->page_size, pool->num_kv_heads};
        sc.trajs = TrajView{reinterpret_cast<const int32_t *>(sb + sl.off_table), reinterpret_cast<const int32_t *>(sb + sl.off_lens),
                            sl.pages_per_item, n_groups};
        sc.traj_ids = nullptr;              // group j is row j of the scratch table
        sc.sm_scale = sm_scale * k_scale;
        sc.v_scale = v_scale;
    }
    e = launch_chunk_attn(sc, stream, &ctx->launches, &too_small);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "group_decode_attn shared-prefix launch");
    // private remainder: the decode kernel over each member's pages after the prefix
    AttnCall pc = base;
    pc.page_offset = item_off;
    pc.out_f32 = part_b;
    pc.lse = lse_b;
    pc.fp8 = fp8;
    pc.k_scale = k_scale;
    pc.v_scale = v_scale;
    e = launch_decode_attn(pc, stream, &ctx->launches, &too_small);
    if (too_small) return fail(ctx, ROLLART_ERR_WORKSPACE, "workspace of %zu bytes is too small", ctx->workspace_bytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "group_decode_attn decode launch");
    e = launch_group_merge(part_a, lse_a, part_b, lse_b, static_cast<long long>(n_items) * num_q_heads,
                           static_cast<__nv_bfloat16 *>(out), lse, stream, &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "group_decode_attn merge launch");
    return ROLLART_OK;
}

rollart_status rollart_group_decode_attn(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                         const int32_t *traj_ids, int32_t n_items, const int32_t *group_indptr,
                                         const int32_t *shared_lens, int32_t n_groups, int32_t max_seq_len, const void *q,
                                         int32_t num_q_heads, float sm_scale, void *out, float *lse, void *stream) {
    return group_decode_impl(ctx, pool, trajs, traj_ids, n_items, group_indptr, shared_lens, n_groups, max_seq_len, q,
                             num_q_heads, sm_scale, out, lse, stream, false, 1.f, 1.f, nullptr, 0);
}

rollart_status rollart_group_decode_attn_fp8(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                             const int32_t *traj_ids, int32_t n_items, const int32_t *group_indptr,
                                             const int32_t *shared_lens, int32_t n_groups, int32_t max_seq_len, const void *q,
                                             int32_t num_q_heads, float sm_scale, float k_scale, float v_scale, void *out,
                                             float *lse, void *scratch, size_t scratch_bytes, void *stream) {
    return group_decode_impl(ctx, pool, trajs, traj_ids, n_items, group_indptr, shared_lens, n_groups, max_seq_len, q,
                             num_q_heads, sm_scale, out, lse, stream, true, k_scale, v_scale, scratch, scratch_bytes);
}

rollart_status rollart_obs_chunk_attn(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                      const int32_t *traj_ids, const int32_t *q_indptr, int32_t n_items,
                                      int32_t total_q, int32_t max_seq_len, const void *q, int32_t num_q_heads,
                                      float sm_scale, void *out, float *lse, void *stream) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    rollart_status st = attn_common(ctx, pool, trajs, n_items, total_q, max_seq_len, q, num_q_heads, out);
    if (st != ROLLART_OK) return st;
    if (n_items == 0 || total_q == 0) return ROLLART_OK;
    if (!q_indptr) return fail(ctx, ROLLART_ERR_INVALID_ARG, "q_indptr NULL");
    max_seq_len = clamp_bound(pool, trajs, max_seq_len);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, ROLLART_ERR_CUDA, "cannot select device %d", ctx->device);
    AttnCall c = make_call(ctx, pool, trajs, traj_ids, q_indptr, n_items, total_q, max_seq_len, q, num_q_heads, sm_scale,
                           out, lse);
    bool too_small = false;
    cudaError_t e = launch_chunk_attn(c, static_cast<cudaStream_t>(stream), &ctx->launches, &too_small);
    if (too_small) return fail(ctx, ROLLART_ERR_WORKSPACE, "workspace of %zu bytes is too small", ctx->workspace_bytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "obs_chunk_attn launch");
    return ROLLART_OK;
}

size_t rollart_obs_chunk_fp8_scratch_size(int32_t n_items, int32_t num_kv_heads, int32_t page_size, int32_t max_seq_len) {
    if (n_items <= 0 || num_kv_heads <= 0 || page_size <= 0 || max_seq_len < 0) return 0;
    return fp8_chunk_scratch_bytes(n_items, num_kv_heads, page_size, max_seq_len, -1);
}

size_t rollart_obs_chunk_fp8_scratch_size_for_pages(int32_t n_items, int32_t num_kv_heads, int32_t page_size,
                                                    int32_t max_seq_len, int64_t total_pages) {
    if (n_items <= 0 || num_kv_heads <= 0 || page_size <= 0 || max_seq_len < 0 || total_pages < 0) return 0;
    return fp8_chunk_scratch_bytes(n_items, num_kv_heads, page_size, max_seq_len, total_pages);
}

rollart_status rollart_obs_chunk_attn_fp8(rollart_ctx *ctx, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                          const int32_t *traj_ids, const int32_t *q_indptr, int32_t n_items,
                                          int32_t total_q, int32_t max_seq_len, const void *q, int32_t num_q_heads,
                                          float sm_scale, float k_scale, float v_scale, void *out, float *lse,
                                          void *scratch, size_t scratch_bytes, void *stream) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    rollart_status st = attn_common(ctx, pool, trajs, n_items, total_q, max_seq_len, q, num_q_heads, out);
    if (st != ROLLART_OK) return st;
    if (!(k_scale > 0.f) || !(v_scale > 0.f) || !isfinite(k_scale) || !isfinite(v_scale))
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "k_scale and v_scale must be positive and finite");
    if (n_items == 0 || total_q == 0) return ROLLART_OK;
    if (!q_indptr) return fail(ctx, ROLLART_ERR_INVALID_ARG, "q_indptr NULL");
    max_seq_len = clamp_bound(pool, trajs, max_seq_len);
    const Fp8ChunkScratch L = fp8_chunk_scratch_layout(n_items, pool->num_kv_heads, pool->page_size, max_seq_len, scratch_bytes);
    if (!scratch || (reinterpret_cast<uintptr_t>(scratch) & 255u) != 0)
        return fail(ctx, ROLLART_ERR_INVALID_ARG, "scratch must be a 256-byte aligned device buffer");
    if (L.capacity_pages < 1)
        return fail(ctx, ROLLART_ERR_WORKSPACE, "scratch of %zu bytes cannot hold a single page", scratch_bytes);
    if (static_cast<long long>(n_items) * L.pages_per_item > 0x7FFFFFFFLL)
        return fail(ctx, ROLLART_ERR_UNSUPPORTED, "too many scratch pages");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, ROLLART_ERR_CUDA, "cannot select device %d", ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = launch_fp8_pages_to_bf16(*pool, *trajs, traj_ids, nullptr, n_items, max_seq_len, L, scratch, ctx->d_status, s,
                                             &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "fp8 expansion launch");
    // the attention itself runs over the expanded copy: item i is row i of the scratch table
    char *base = static_cast<char *>(scratch);
    rollart_kv_pool spool = *pool;
    spool.k_pool = base + L.off_k;
    spool.v_pool = base + L.off_v;
    spool.num_pages = static_cast<int32_t>(L.capacity_pages);
    rollart_trajs strajs;
    strajs.page_table = reinterpret_cast<const int32_t *>(base + L.off_table);
    strajs.max_pages_per_traj = L.pages_per_item;
    strajs.seq_lens = reinterpret_cast<const int32_t *>(base + L.off_lens);
    strajs.num_traj = n_items;
    AttnCall c = make_call(ctx, &spool, &strajs, nullptr, q_indptr, n_items, total_q, max_seq_len, q, num_q_heads,
                           sm_scale * k_scale, out, lse);
    c.v_scale = v_scale;
    bool too_small = false;
    e = launch_chunk_attn(c, s, &ctx->launches, &too_small);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "obs_chunk_attn launch");
    return ROLLART_OK;
}

rollart_status rollart_selftest_bounded_wait(rollart_ctx *ctx, void *stream) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, ROLLART_ERR_CUDA, "cannot select device %d", ctx->device);
    cudaError_t e = launch_bounded_wait_selftest(ctx->d_status, static_cast<cudaStream_t>(stream), &ctx->launches);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "bounded-wait self-test launch");
    return ROLLART_OK;
}

rollart_status rollart_check(rollart_ctx *ctx, void *stream) {
    if (!ctx) return ROLLART_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, ROLLART_ERR_CUDA, "cannot select device %d", ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(ctx->h_status, ctx->d_status, sizeof(DeviceStatus), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_status, 0, sizeof(DeviceStatus), s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "rollart_check");
    const DeviceStatus hs = *ctx->h_status;
    if (hs.code == 0) return ROLLART_OK;
    decode_reset_workspace(ctx->workspace, ctx->workspace_bytes, s);
    cudaStreamSynchronize(s);
    static const char *const where[] = {"?", "kv_append", "decode_attn", "obs_chunk_attn", "combine", "kv_gather", "pages",
                                        "group_decode"};
    const char *w = (hs.where >= 0 && hs.where < 8) ? where[hs.where] : "?";
    if (hs.code == ROLLART_ERR_TIMEOUT)
        return fail(ctx, ROLLART_ERR_TIMEOUT, "%s: a bounded wait ran out (detail %d)", w, hs.detail);
    if (hs.code == ROLLART_ERR_WORKSPACE)
        return fail(ctx, ROLLART_ERR_WORKSPACE, "%s: the scratch buffer is smaller than the contexts listed (item %d)", w, hs.detail);
    return fail(ctx, static_cast<rollart_status>(hs.code), "%s: index out of range on the device (detail %d)", w, hs.detail);
}

const char *rollart_last_error(rollart_ctx *ctx) { return ctx ? ctx->err : "context is NULL"; }

int64_t rollart_launch_count(rollart_ctx *ctx) { return ctx ? ctx->launches : 0; }

}  // extern "C"
