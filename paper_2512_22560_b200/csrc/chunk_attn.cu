// Observation-chunk attention on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// Work unit: (item, kv head, M-tile).  An M-tile is 128 query rows = floor(128 / g) consecutive
// chunk tokens x the g query heads that share the kv head, so one K/V read serves all of them.
// The unit walks the visible keys (the whole cached prefix, then the chunk itself up to the
// diagonal) in tiles of 64 keys:
//
//   S = Q K^T      tcgen05.mma, M 128 x N 64 x K 128, operands in 128B-swizzled shared memory
//                  (Q and K tiles brought by TMA), fp32 accumulator in TMEM, double buffered
//   softmax        one thread per query row (4 warps = 128 TMEM lanes): tcgen05.ld its 64 scores,
//                  scale, causal/length mask, running max m and sum l, P = exp2(s - m) as packed
//                  bf16 stored back with tcgen05.st over the first 32 columns of the same S
//                  buffer; the O accumulator in TMEM is rescaled only when a row's max has grown
//                  by more than 2^8, so the softmax warps normally never wait for an MMA
//   O += P V       tcgen05.mma with the A operand (P) in TMEM, M 128 x N 128 x K 64; V is the
//                  MN-major B operand straight from its [key][dim] page layout
//
// One warp issues the copies, one warp issues the MMAs, four warps do softmax and the epilogue.
// A block uses 97 KB of shared memory and 256 TMEM columns, so two blocks share an SM and one
// block's softmax overlaps the other's MMAs.  Blocks are ordered (item, kv head, M-tile), so the
// M-tiles that re-read one (item, head)'s keys run together and find them in L2.
// Every wait is a bounded mbarrier poll; no block waits for another block.
#include <cuda.h>

#include "rollart_internal.cuh"

namespace rollart {

namespace {

constexpr int kRows = 128;                 // query rows of an M-tile (UMMA M)
constexpr int kKeys = 64;                  // keys per KV tile
constexpr int kStages = 2;
constexpr int kThreads = 192;              // warp 0 copies, warp 1 MMA, warps 2-5 softmax
constexpr int kMaxItems = 1024;            // items per launch (tile prefix lives in shared memory)
constexpr uint32_t kSpinLimit = 1u << 17;   // polls per wait; each poll sleeps in hardware for up to kSuspendNs
constexpr uint32_t kSuspendNs = 10000;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.f;   // log2 units

constexpr int kHalfQ = kRows * 128;        // 16 KB: 128 rows x 64 dims
constexpr int kHalfKV = kKeys * 128;       // 8 KB: 64 keys x 64 dims
constexpr int kOffQ = 0;                                   // [half][row][128 B]
constexpr int kOffK = kOffQ + 2 * kHalfQ;                  // stages x [half][key][128 B]
constexpr int kOffV = kOffK + kStages * 2 * kHalfKV;
constexpr int kOffBars = kOffV + kStages * 2 * kHalfKV;
constexpr int kNumBars = 1 + 4 * kStages + 2 + 2 + 2;      // q | k,v full/empty | s_full x2 | p_full x2 | o_done x2
constexpr int kOffTmemSlot = kOffBars + kNumBars * 8;
constexpr int kOffAbort = kOffTmemSlot + 8;
constexpr int kSmemUsed = kOffAbort + 8;
constexpr int kSmemBytes = kSmemUsed + 1024;               // + slack for the 1024-byte alignment; two blocks fit an SM
static_assert(2 * (kSmemBytes + 1024) <= 228 * 1024, "two blocks per SM");
static_assert((kMaxItems + 1) * 4 <= kStages * 2 * kHalfKV, "the tile prefix is staged in the K stages");

constexpr int kTmemCols = 256;             // S0 [0,64) S1 [64,128) O [128,256); P overwrites the first 32 columns of its S

struct ChunkParams {
    const int32_t *page_table;
    const int32_t *seq_lens;
    const int32_t *traj_ids;
    const int32_t *q_indptr;
    int max_pages, num_traj, num_pages, page_size, num_kv_heads, num_q_heads, group;
    int n_items, item_offset, max_seq_len, total_q;
    __nv_bfloat16 *out;
    float *lse;
    float scale_log2;
    // shared-prefix mode (NULL otherwise): every row of item i sees exactly the first shared_lens[i] keys, no causal mask
    const int32_t *shared_lens;
    float *out_f32;             // when set, result rows go here in fp32 instead of bf16 to `out`
    DeviceStatus *status;
};

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(kSuspendNs) : "memory");
    return ok != 0;
}
// Bounded wait; once any thread of the block has given up, nobody waits any more, so every role
// runs its (bounded) loops to the end and the block exits with the error recorded.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, DeviceStatus *status,
                                          int where) {
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return;
        if (*abort_flag) return;
    }
    if (*abort_flag == 0) {
        *abort_flag = 1;
        report(status, ROLLART_ERR_TIMEOUT, where, 3);
        status->fatal = 1;         // later blocks of this launch do not start
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc], issued by one thread
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// same with the A operand in TMEM (lane = row, packed 16-bit pairs along the columns)
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// the mbarrier gets one arrival when every MMA issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
          "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]),
          "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// three-input max and two-wide fp32 FMA / ADD: half the instructions of the scalar forms
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float min3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ void fma2(float &d0, float &d1, float a0, float a1, float b, float c) {   // d = a * b + c, two lanes
    asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\tmov.b64 rc, {%5, %5};\n\t"
        "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b), "f"(c));
}
__device__ __forceinline__ void add2(float &d0, float &d1, float a0, float a1) {                      // d += a, two lanes
    asm("{\n\t.reg .b64 ra, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rd, {%0, %1};\n\t"
        "add.rn.f32x2 rd, rd, ra;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "+f"(d0), "+f"(d1) : "f"(a0), "f"(a1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Shared-memory matrix descriptor of a 128B-swizzled operand tile whose 8-row groups are 1024 B
// apart (stride byte offset); `lbo` is the distance between 64-element blocks along the
// contiguous dimension of an MN-major operand (ignored for K-major tiles, where it is set to 16).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo) {
    return static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(lbo >> 4) << 16) |
           (static_cast<uint64_t>(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, A K-major, M = 128.
constexpr uint32_t idesc(int n, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | (static_cast<uint32_t>(n >> 3) << 17) |
           (static_cast<uint32_t>(kRows >> 4) << 24);
}

// ------------------------------------------------------------------------------------------
// Kernel
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 2)
chunk_attn_kernel(const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap kmap,
                  const __grid_constant__ CUtensorMap vmap, const ChunkParams prm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hkv = prm.num_kv_heads, P = prm.page_size, g = prm.group;
    const int tpt = kRows / g;                       // chunk tokens per M-tile
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + kOffAbort);
    volatile uint32_t *s_tmem = reinterpret_cast<volatile uint32_t *>(smem + kOffTmemSlot);
    int *s_prefix = reinterpret_cast<int *>(smem + kOffK);     // staged in the K stages during the prologue

    if (static_cast<int>(smem - smem_raw) + kSmemUsed > kSmemBytes) {   // cannot happen: the slack covers any alignment
        if (threadIdx.x == 0) report(prm.status, ROLLART_ERR_CUDA, static_cast<int>(smem - smem_raw), 3);
        return;
    }
    const uint32_t bars = smem_u32(smem + kOffBars);
    const uint32_t bar_q = bars;
    auto bar_kfull = [&](int s) { return bars + 8u * (1 + s); };
    auto bar_kempty = [&](int s) { return bars + 8u * (1 + kStages + s); };
    auto bar_vfull = [&](int s) { return bars + 8u * (1 + 2 * kStages + s); };
    auto bar_vempty = [&](int s) { return bars + 8u * (1 + 3 * kStages + s); };
    auto bar_sfull = [&](int s) { return bars + 8u * (1 + 4 * kStages + s); };
    // tile i uses p_full(i & 1) and o_done(i & 1): a warp that is a tile ahead of the others arrives on the other barrier
    auto bar_pfull = [&](int s) { return bars + 8u * (1 + 4 * kStages + 2 + s); };
    auto bar_odone = [&](int s) { return bars + 8u * (1 + 4 * kStages + 4 + s); };

    // ---- which (item, kv head, M-tile) is this block?  tiles per item -> prefix -> search ----
    for (int i = threadIdx.x; i < prm.n_items; i += kThreads) {
        const int n = __ldg(prm.q_indptr + i + 1) - __ldg(prm.q_indptr + i);
        s_prefix[i + 1] = n > 0 ? (n + tpt - 1) / tpt : 0;
    }
    if (threadIdx.x == 0) {
        s_prefix[0] = 0;
        mbar_init(bar_q, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_kfull(s), 1); mbar_init(bar_kempty(s), 1);
            mbar_init(bar_vfull(s), 1); mbar_init(bar_vempty(s), 1);
        }
        for (int s = 0; s < 2; ++s) { mbar_init(bar_sfull(s), 1); mbar_init(bar_odone(s), 1); mbar_init(bar_pfull(s), 4); }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (warp == 0) {        // inclusive scan of the tile counts, in place
        const int per = (prm.n_items + 31) / 32;
        const int a = min(prm.n_items, lane * per), b = min(prm.n_items, a + per);
        int sum = 0;
        for (int i = a; i < b; ++i) sum += s_prefix[i + 1];
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        int run = incl - sum;
        for (int i = a; i < b; ++i) { run += s_prefix[i + 1]; s_prefix[i + 1] = run; }
    }
    __syncthreads();
    const int unit = blockIdx.x;
    const int total_units = s_prefix[prm.n_items] * hkv;
    int item = 0, head = 0, mtile = 0;
    if (unit < total_units) {
        int lo = 0, hi = prm.n_items;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_prefix[mid] * hkv <= unit) lo = mid; else hi = mid;
        }
        item = lo;
        const int nt = max(1, s_prefix[lo + 1] - s_prefix[lo]);
        const int rem = unit - s_prefix[lo] * hkv;
        head = rem / nt;
        mtile = nt - 1 - (rem - head * nt);     // later M-tiles see more keys: start the longest ones first
    }
    __syncthreads();                 // everyone has read the prefix: the K stages are free again
    if (unit >= total_units) return;
    if (*reinterpret_cast<volatile int *>(&prm.status->fatal) != 0) return;   // an earlier block ran out of patience: give up quickly

    // ---- geometry of this unit ----
    const bool shared_mode = prm.shared_lens != nullptr;
    const int q_row0 = __ldg(prm.q_indptr + item);
    const int n_chunk = __ldg(prm.q_indptr + item + 1) - q_row0;
    const int t = prm.traj_ids ? __ldg(prm.traj_ids + item) : item + prm.item_offset;
    int L = 0;
    bool bad = false;
    if (q_row0 < 0 || n_chunk < 0 || static_cast<long long>(q_row0) + n_chunk > prm.total_q) {
        bad = true;                  // q_indptr does not describe rows of q
        if (threadIdx.x == 0) report(prm.status, ROLLART_ERR_BOUNDS, q_row0, 3);
    } else if (t < 0 || t >= prm.num_traj) {
        bad = true;
        if (threadIdx.x == 0) report(prm.status, ROLLART_ERR_BOUNDS, t, 3);
    } else {
        L = __ldg(prm.seq_lens + t);
        if (shared_mode) {
            const int s_len = __ldg(prm.shared_lens + item);
            if (s_len < 0 || s_len > L) {
                bad = true;
                if (threadIdx.x == 0) report(prm.status, ROLLART_ERR_BOUNDS, s_len, 3);
            }
            L = s_len;               // keys beyond the shared prefix do not exist for this call
        }
        if (!bad && (L < 0 || L > prm.max_seq_len || (!shared_mode && n_chunk > L))) {
            bad = true;
            if (threadIdx.x == 0) report(prm.status, ROLLART_ERR_BOUNDS, L, 3);
        }
    }
    if (bad) return;                 // uniform over the block, before any barrier or TMEM use
    const int prior = L - n_chunk;
    const int tok0 = mtile * tpt;                              // first chunk token of this M-tile
    const int toks = min(tpt, n_chunk - tok0);                 // live tokens
    const int max_count = shared_mode ? L : prior + tok0 + toks;   // keys visible to the last live row
    const int min_count = shared_mode ? L : prior + tok0 + 1;      // keys visible to the first row
    const int n_tiles = (max_count + kKeys - 1) / kKeys;
    const int32_t *table_row = prm.page_table + static_cast<long long>(t) * prm.max_pages;
    if (n_tiles == 0) {
        // only in shared-prefix mode with an empty prefix: the result is out = 0, lse = -inf
        for (int idx = threadIdx.x; idx < toks * g * (kHeadDim / 4); idx += kThreads) {
            const int r = idx / (kHeadDim / 4), c = idx - r * (kHeadDim / 4);
            const int tk = r / g, hd = r - tk * g;
            const long long orow = static_cast<long long>(q_row0 + tok0 + tk) * prm.num_q_heads + head * g + hd;
            if (prm.out_f32 != nullptr) reinterpret_cast<float4 *>(prm.out_f32 + orow * kHeadDim)[c] = make_float4(0.f, 0.f, 0.f, 0.f);
            else reinterpret_cast<uint2 *>(prm.out + orow * kHeadDim)[c] = make_uint2(0u, 0u);
            if (c == 0 && prm.lse != nullptr) prm.lse[orow] = -INFINITY;
        }
        return;                      // uniform over the block, before any barrier or TMEM use
    }

    // zero the Q tile (rows beyond tpt * g are never written by the copy) and allocate TMEM
    for (int i = threadIdx.x; i < 2 * kHalfQ / 16; i += kThreads) reinterpret_cast<uint4 *>(smem + kOffQ)[i] = make_uint4(0, 0, 0, 0);
    fence_proxy_async();
    if (warp == 0) tmem_alloc(smem_u32(smem + kOffTmemSlot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *s_tmem;

    if (warp == 0) {
        // =============================== copy warp ===============================
        if (lane == 0) {
            mbar_arrive_expect_tx(bar_q, static_cast<uint32_t>(tpt * g) * kRowBytes);
            tma_load_3d(smem_u32(smem + kOffQ), &qmap, bar_q, 0, head * g, q_row0 + tok0);
            tma_load_3d(smem_u32(smem + kOffQ + kHalfQ), &qmap, bar_q, 64, head * g, q_row0 + tok0);
        }
        const int pages_per_tile = kKeys / P;
        const uint32_t half_page = static_cast<uint32_t>(P) * 128;
        for (int j = 0; j < n_tiles; ++j) {
            const int stage = j % kStages;
            const uint32_t par = ((j / kStages) & 1) ^ 1;
            const int lp = j * pages_per_tile + lane;
            int pg = -1;
            if (lane < pages_per_tile && lp * P < L) {
                pg = __ldg(table_row + lp);
                if (pg < 0 || pg >= prm.num_pages) { report(prm.status, ROLLART_ERR_BOUNDS, pg, 3); pg = -1; }
            }
            const uint32_t nvalid = __popc(__ballot_sync(0xffffffffu, pg >= 0));
            const int row = (pg * hkv + head) * P;
            // K
            mbar_wait(bar_kempty(stage), par, s_abort, prm.status, 1);
            if (!*s_abort) {
                if (lane == 0) mbar_arrive_expect_tx(bar_kfull(stage), nvalid * 2u * half_page);
                __syncwarp();
                if (pg >= 0) {
                    const uint32_t dst = smem_u32(smem + kOffK + stage * 2 * kHalfKV) + lane * half_page;
                    tma_load_2d(dst, &kmap, bar_kfull(stage), 0, row);
                    tma_load_2d(dst + kHalfKV, &kmap, bar_kfull(stage), 64, row);
                }
            }
            // V
            mbar_wait(bar_vempty(stage), par, s_abort, prm.status, 2);
            if (!*s_abort) {
                if (lane == 0) mbar_arrive_expect_tx(bar_vfull(stage), nvalid * 2u * half_page);
                __syncwarp();
                if (pg >= 0) {
                    const uint32_t dst = smem_u32(smem + kOffV + stage * 2 * kHalfKV) + lane * half_page;
                    tma_load_2d(dst, &vmap, bar_vfull(stage), 0, row);
                    tma_load_2d(dst + kHalfKV, &vmap, bar_vfull(stage), 64, row);
                }
            }
        }
    } else if (warp == 1) {
        // =============================== MMA warp ===============================
        constexpr uint32_t kIdescQK = idesc(kKeys, false);
        constexpr uint32_t kIdescPV = idesc(kHeadDim, true);
        const uint32_t q_addr = smem_u32(smem + kOffQ);
        auto issue_pv = [&](int i) {
            const int stage = i % kStages;
            mbar_wait(bar_vfull(stage), (i / kStages) & 1, s_abort, prm.status, 3);
            mbar_wait(bar_pfull(i & 1), (i >> 1) & 1, s_abort, prm.status, 4);
            tc_fence_after();
            if (lane == 0 && !*s_abort) {
                const uint32_t v_addr = smem_u32(smem + kOffV + stage * 2 * kHalfKV);
#pragma unroll
                for (int ks = 0; ks < kKeys / 16; ++ks)   // 16 keys per step: 8 packed columns along P's row, 2048 B down V
                    umma_bf16_ts(tmem + 128, tmem + (i & 1) * kKeys + ks * 8, smem_desc(v_addr + ks * 2048, kHalfKV), kIdescPV,
                                 (i > 0 || ks > 0) ? 1u : 0u);
                umma_commit(bar_vempty(stage));
                umma_commit(bar_odone(i & 1));
            }
            __syncwarp();
        };
        mbar_wait(bar_q, 0, s_abort, prm.status, 5);
        for (int j = 0; j < n_tiles; ++j) {
            const int stage = j % kStages, sb = j & 1;
            mbar_wait(bar_kfull(stage), (j / kStages) & 1, s_abort, prm.status, 6);
            // S buffer sb last held P of tile j-2; PV(j-2) was issued before this QK and MMAs run in issue order
            tc_fence_after();
            if (lane == 0 && !*s_abort) {
                const uint32_t k_addr = smem_u32(smem + kOffK + stage * 2 * kHalfKV);
#pragma unroll
                for (int ks = 0; ks < kHeadDim / 16; ++ks) {   // 16 dims per step; the second 64 dims live in the other half
                    const uint32_t qa = q_addr + (ks >> 2) * kHalfQ + (ks & 3) * 32;
                    const uint32_t ka = k_addr + (ks >> 2) * kHalfKV + (ks & 3) * 32;
                    umma_bf16(tmem + sb * kKeys, smem_desc(qa, 16), smem_desc(ka, 16), kIdescQK, ks > 0 ? 1u : 0u);
                }
                umma_commit(bar_kempty(stage));
                umma_commit(bar_sfull(sb));
            }
            __syncwarp();
            if (j >= 1) issue_pv(j - 1);
        }
        issue_pv(n_tiles - 1);
    } else {
        // =============================== softmax warps ===============================
        const int quarter = warp & 3;                         // TMEM lanes 32 * quarter .. + 31 belong to this warp
        const int row = quarter * 32 + lane;
        const uint32_t lane_addr = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        const int tok_local = row / g, head_local = row - tok_local * g;
        const bool live = tok_local < toks;
        const int count = shared_mode ? L : min(L, prior + tok0 + min(tok_local, toks - 1) + 1);   // keys this row sees (>= 1)
        float m_ref = -INFINITY, l_sum = 0.f;

        for (int j = 0; j < n_tiles; ++j) {
            const int sb = j & 1;
            mbar_wait(bar_sfull(sb), (j >> 1) & 1, s_abort, prm.status, 8);
            tc_fence_after();
            uint32_t sraw[2][32];
            tmem_ld32(lane_addr + sb * kKeys, sraw[0]);
            tmem_ld32(lane_addr + sb * kKeys + 32, sraw[1]);
            tmem_wait_ld();

            const int key0 = j * kKeys;
            const bool need_mask = key0 + kKeys > min_count;    // uniform over the block
            const float scale = prm.scale_log2;
            float rmax;
            if (!need_mask) {
                // the max of scale * s is scale * (max or min of s): take the extreme of the raw scores, 8 chains of 3-input ops
                float e[8];
                if (scale >= 0.f) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) e[k] = max3(__uint_as_float(sraw[0][k]), __uint_as_float(sraw[0][8 + k]), __uint_as_float(sraw[0][16 + k]));
#pragma unroll
                    for (int k = 0; k < 8; ++k) e[k] = max3(e[k], __uint_as_float(sraw[0][24 + k]), __uint_as_float(sraw[1][k]));
#pragma unroll
                    for (int k = 0; k < 8; ++k) e[k] = max3(e[k], __uint_as_float(sraw[1][8 + k]), __uint_as_float(sraw[1][16 + k]));
#pragma unroll
                    for (int k = 0; k < 8; ++k) e[k] = fmaxf(e[k], __uint_as_float(sraw[1][24 + k]));
                    rmax = max3(max3(e[0], e[1], e[2]), max3(e[3], e[4], e[5]), fmaxf(e[6], e[7])) * scale;
                } else {
#pragma unroll
                    for (int k = 0; k < 8; ++k) e[k] = min3(__uint_as_float(sraw[0][k]), __uint_as_float(sraw[0][8 + k]), __uint_as_float(sraw[0][16 + k]));
#pragma unroll
                    for (int k = 0; k < 8; ++k) e[k] = min3(e[k], __uint_as_float(sraw[0][24 + k]), __uint_as_float(sraw[1][k]));
#pragma unroll
                    for (int k = 0; k < 8; ++k) e[k] = min3(e[k], __uint_as_float(sraw[1][8 + k]), __uint_as_float(sraw[1][16 + k]));
#pragma unroll
                    for (int k = 0; k < 8; ++k) e[k] = fminf(e[k], __uint_as_float(sraw[1][24 + k]));
                    rmax = min3(min3(e[0], e[1], e[2]), min3(e[3], e[4], e[5]), fminf(e[6], e[7])) * scale;
                }
            } else {
                rmax = -INFINITY;
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (key0 + h * 32 + c < count) rmax = fmaxf(rmax, __uint_as_float(sraw[h][c]) * scale);
            }
            // the reference max moves only when it has to (first tile) or when a row outgrew it by 2^8
            const bool grow = rmax > m_ref + kRescaleThreshold;
            const float m_new = grow ? rmax : m_ref;
            const float corr = grow ? ex2(m_ref - m_new) : 1.f;   // ex2(-inf) = 0 on the first tile
            const float neg_m = -m_new;
            float rs[4] = {0.f, 0.f, 0.f, 0.f};
            uint32_t packed[32];
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                    float x0, x1;
                    fma2(x0, x1, __uint_as_float(sraw[h][c]), __uint_as_float(sraw[h][c + 1]), scale, neg_m);
                    float p0 = ex2(x0), p1 = ex2(x1);
                    if (need_mask) {
                        p0 = key0 + h * 32 + c < count ? p0 : 0.f;
                        p1 = key0 + h * 32 + c + 1 < count ? p1 : 0.f;
                    }
                    add2(rs[c & 2], rs[(c & 2) + 1], p0, p1);
                    packed[h * 16 + (c >> 1)] = pack_bf16(p0, p1);
                }
            const float rsum = (rs[0] + rs[1]) + (rs[2] + rs[3]);
            l_sum = l_sum * corr + rsum;
            m_ref = m_new;

            if (j >= 1 && __any_sync(0xffffffffu, grow)) {
                // rare: some row of this warp moved its reference max, so O (tiles 0 .. j-1) must be rescaled
                // before PV of this tile; PV of tile j-1 has to be finished first
                mbar_wait(bar_odone((j - 1) & 1), ((j - 1) >> 1) & 1, s_abort, prm.status, 9);
                tc_fence_after();
#pragma unroll 1
                for (int c0 = 0; c0 < kHeadDim; c0 += 32) {
                    uint32_t oraw[32];
                    tmem_ld32(lane_addr + 128 + c0, oraw);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 32; ++c) oraw[c] = __float_as_uint(__uint_as_float(oraw[c]) * corr);
                    tmem_st32(lane_addr + 128 + c0, oraw);
                }
            }
            // P as the next A operand: 64 bf16 of this row as 32 packed columns over the start of its S buffer
            tmem_st32(lane_addr + sb * kKeys, packed);
            tmem_wait_st();
            if (key0 + kKeys > L) {
                // keys at or beyond L are dead slots (or were never copied): their V rows must be 0, not garbage
                mbar_wait(bar_vfull(j % kStages), (j / kStages) & 1, s_abort, prm.status, 10);
                const uint32_t v_addr = smem_u32(smem + kOffV + (j % kStages) * 2 * kHalfKV);
                const int first_dead = L - key0;
                for (int idx = threadIdx.x - 64; idx < (kKeys - first_dead) * 16; idx += 128) {
                    const int r = first_dead + (idx >> 4), c = idx & 15;
                    asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(v_addr + (c >> 3) * kHalfKV + r * 128 + (c & 7) * 16),
                                 "r"(0) : "memory");
                }
                fence_proxy_async();      // the zeroed V rows become visible to the tensor core's reads
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_pfull(sb));
        }

        // ---- epilogue: O / l -> bf16 rows of out ----
        mbar_wait(bar_odone((n_tiles - 1) & 1), ((n_tiles - 1) >> 1) & 1, s_abort, prm.status, 11);
        tc_fence_after();
        const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
        const long long orow = (static_cast<long long>(q_row0 + tok0 + tok_local) * prm.num_q_heads + head * g + head_local);
#pragma unroll 1
        for (int c0 = 0; c0 < kHeadDim; c0 += 32) {
            uint32_t oraw[32];
            tmem_ld32(lane_addr + 128 + c0, oraw);
            tmem_wait_ld();
            if (live && prm.out_f32 != nullptr) {
                float4 *dst = reinterpret_cast<float4 *>(prm.out_f32 + orow * kHeadDim + c0);
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    dst[k] = make_float4(__uint_as_float(oraw[4 * k]) * inv, __uint_as_float(oraw[4 * k + 1]) * inv,
                                         __uint_as_float(oraw[4 * k + 2]) * inv, __uint_as_float(oraw[4 * k + 3]) * inv);
            } else if (live) {
                uint4 *dst = reinterpret_cast<uint4 *>(prm.out + orow * kHeadDim + c0);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    uint4 v;
                    v.x = pack_bf16(__uint_as_float(oraw[8 * k]) * inv, __uint_as_float(oraw[8 * k + 1]) * inv);
                    v.y = pack_bf16(__uint_as_float(oraw[8 * k + 2]) * inv, __uint_as_float(oraw[8 * k + 3]) * inv);
                    v.z = pack_bf16(__uint_as_float(oraw[8 * k + 4]) * inv, __uint_as_float(oraw[8 * k + 5]) * inv);
                    v.w = pack_bf16(__uint_as_float(oraw[8 * k + 6]) * inv, __uint_as_float(oraw[8 * k + 7]) * inv);
                    dst[k] = v;
                }
            }
        }
        if (live && prm.lse != nullptr) prm.lse[orow] = l_sum > 0.f ? (m_ref + log2f(l_sum)) * kLn2 : -INFINITY;
        tc_fence_before();
    }

    // ---- all roles meet; the allocating warp returns the TMEM columns ----
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// pool as [rows = pages * heads * slots][128 dims]; one box = 64 dims x one page of one head
bool encode_pool_rows(CUtensorMap *map, const void *pool, int num_pages, int hkv, int P) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {kHeadDim, static_cast<cuuint64_t>(num_pages) * hkv * P};
    const cuuint64_t strides[1] = {kRowBytes};
    const cuuint32_t box[2] = {64, static_cast<cuuint32_t>(P)};
    const cuuint32_t ones[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(pool), dims, strides, box, ones,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// q as [token][q head][128 dims]; one box = 64 dims x g heads x (128 / g) tokens, landing as
// [token][head][128 B]: exactly the rows of an M-tile.  Tokens past the end read as zero.
bool encode_q_map(CUtensorMap *map, const void *q, int total_q, int hq, int g) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {kHeadDim, static_cast<cuuint64_t>(hq), static_cast<cuuint64_t>(total_q)};
    const cuuint64_t strides[2] = {kRowBytes, static_cast<cuuint64_t>(hq) * kRowBytes};
    const cuuint32_t box[3] = {64, static_cast<cuuint32_t>(g), static_cast<cuuint32_t>(kRows / g)};
    const cuuint32_t ones[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(q), dims, strides, box, ones,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_chunk_attn(const AttnCall &c, cudaStream_t stream, int64_t *launches, bool *too_small) {
    (void)too_small;
    const int hkv = c.pool.num_kv_heads, g = c.num_q_heads / hkv, tpt = kRows / g;
    cudaError_t e = cudaFuncSetAttribute(chunk_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    CUtensorMap qmap, kmap, vmap;
    if (!encode_q_map(&qmap, c.q, c.total_q, c.num_q_heads, g) ||
        !encode_pool_rows(&kmap, c.pool.k, c.pool.num_pages, hkv, c.pool.page_size) ||
        !encode_pool_rows(&vmap, c.pool.v, c.pool.num_pages, hkv, c.pool.page_size))
        return cudaErrorInvalidValue;
    for (int base = 0; base < c.n_items; base += kMaxItems) {
        const int n = c.n_items - base < kMaxItems ? c.n_items - base : kMaxItems;
        ChunkParams prm;
        prm.page_table = c.trajs.page_table; prm.seq_lens = c.trajs.seq_lens;
        prm.traj_ids = c.traj_ids ? c.traj_ids + base : nullptr;
        prm.q_indptr = c.q_indptr + base;
        prm.max_pages = c.trajs.max_pages; prm.num_traj = c.trajs.num_traj; prm.num_pages = c.pool.num_pages;
        prm.page_size = c.pool.page_size; prm.num_kv_heads = hkv; prm.num_q_heads = c.num_q_heads; prm.group = g;
        prm.n_items = n; prm.item_offset = base; prm.max_seq_len = c.max_seq_len; prm.total_q = c.total_q;
        prm.out = c.out; prm.lse = c.lse; prm.scale_log2 = c.sm_scale * kLog2e; prm.status = c.status;
        prm.shared_lens = c.shared_lens ? c.shared_lens + base : nullptr;
        prm.out_f32 = c.out_f32;
        // an upper bound on the M-tiles of these items: every item has at most one ragged tile
        const long long tiles = (static_cast<long long>(c.total_q) + tpt - 1) / tpt + n;
        const long long blocks = tiles * hkv;
        if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
        chunk_attn_kernel<<<static_cast<unsigned>(blocks), kThreads, kSmemBytes, stream>>>(qmap, kmap, vmap, prm);
        ++*launches;
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace rollart
