// Decode attention: split-KV flash decoding over a paged bf16 KV cache, one persistent thread
// block per SM.
//
// Schedule.  Every (item, kv head) owns ceil(L / 64) key tiles.  All tiles of the call are laid
// on one line, ordered (item, kv head, tile), each (item, head) followed by a few units of padding
// that stand for the fixed cost of working on one more (item, head) (query fetch, the merge of
// the warps, the write-out: 2.7 us measured, four tile times), and the line is cut into gridDim.x
// equal spans, one per thread block.  A block therefore has the same work as every other block
// whatever the length mix, and a span that crosses an (item, head) boundary simply starts a new
// "piece".  A piece that covers its (item, head) entirely writes the final bf16 output; otherwise
// it writes an un-normalised fp32 partial (O, m, l) into a workspace slot and takes a ticket; the
// block that takes the last ticket of an (item, head) merges all its slots, in block order, with
// the log-sum-exp rule (cross-split combine) and writes the output.  The cut and the merge order
// are fixed functions of the lengths, so reruns are bit identical.
//
// Data path.  Two producer warps (one for K and the queries, one for V) walk the block's span and
// bring each 64-key tile of K and V (32 KB) into a ring of shared-memory stages with TMA tensor copies, one box per (page, head)
// (or per half row), 128-byte swizzled so that ldmatrix reads are bank-conflict free; the page
// ids come from the page table a batch ahead of the copies.  Eight consumer warps in two groups take
// alternate tiles; each warp owns 16 keys of a tile and computes, for all (up to 16) query heads
// of the GQA group at once, S = Q K^T and O += P V with bf16 mma.sync (fp32 accumulate) and an
// online softmax in registers.  One K/V read serves the whole group.  At the end of a piece the
// eight warps merge into a double-buffered shared tile and go straight on to the next piece; a
// tenth warp writes the tile out (output or slot), takes the ticket and does the combine, off
// the consumers' critical path.  HBM traffic is the KV bytes once, plus Q, O and the few slots.
#include <cuda.h>

#include <cstdarg>
#include <cstdio>
#include <mutex>

#include "rollart_internal.cuh"

namespace rollart {

namespace {

constexpr int kTile = 64;                 // keys per stage
constexpr int kPieceCost = 4;             // what starting another (item, head) costs a block, in tile times (measured: 2.7 us)
constexpr int kStages = 6;
constexpr int kConsumerWarps = 8;         // two groups of four
constexpr int kProducerWarp = kConsumerWarps;        // warp 8 issues the copies
constexpr int kEpilogueWarp = kConsumerWarps + 1;    // warp 9 writes pieces out and combines splits
constexpr int kProducerWarpV = kConsumerWarps + 2;   // warp 10 issues the V copies (warp 8 the K copies and Q)
constexpr int kThreads = (kConsumerWarps + 3) * 32;
constexpr int kThreadsFp8 = kThreads;
constexpr int kMaxItems = 512;            // items per launch (prefix table lives in shared memory)
constexpr int kTensorBytes = kTile * kRowBytes;      // 16 KB of K (or V) per stage
constexpr int kStageBytes = 2 * kTensorBytes;
constexpr int kQBytes = kMaxGroup * kRowBytes;       // 4 KB
constexpr int kMergeStride = kHeadDim + 8;           // floats per merge-buffer row (padded)
constexpr uint32_t kSpinLimit = 1u << 17;   // polls of the drain loop that runs once a block has given up
constexpr long long kWaitCycles = 2000000000LL;   // a wait gives up after about a second
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr size_t kSlotFloats = kMaxGroup * kHeadDim + 2 * kMaxGroup;

// shared-memory map (offsets from a 1024-byte aligned base)
constexpr int kOffStages = 0;
constexpr int kOffQ = kOffStages + kStages * kStageBytes;
constexpr int kOffMerge = kOffQ + 2 * kQBytes;
constexpr int kMergeFloats = kMaxGroup * kMergeStride;              // one merge buffer; there are two
constexpr int kMlFloats = kConsumerWarps * kMaxGroup * 2;           // (m, l) of every warp and row; two copies
constexpr int kOffMl = kOffMerge + 2 * kMergeFloats * 4;
constexpr int kOffLens = kOffMl + 2 * kMlFloats * 4;
constexpr int kOffPrefix = kOffLens + kMaxItems * 4;
constexpr int kOffTraj = kOffPrefix + (kMaxItems + 32) * 4;   // trajectory of every item (read once from global memory)
constexpr int kOffBars = kOffTraj + kMaxItems * 4;
constexpr int kNumBars = 2 * kStages + 8;
constexpr int kOffAbort = kOffBars + kNumBars * 8;
constexpr int kSmemBytes = kOffAbort + 16 + 1024;    // + slack for the 1024-byte alignment
static_assert(kSmemBytes <= 227 * 1024, "the block must fit the shared memory of an SM");

struct DecodeParams {
    const int32_t *page_table;
    const int32_t *seq_lens;
    const int32_t *traj_ids;
    int max_pages, num_traj, num_pages, page_size, num_kv_heads, num_q_heads, group;
    int n_items, item_offset, max_seq_len;
    int four_d;                 // tensor maps are 4-D (one box per page) instead of 2-D (two boxes)
    const __nv_bfloat16 *q;
    __nv_bfloat16 *out;
    float *lse;
    float scale_log2;           // sm_scale * log2(e) (times the K scale of an fp8 pool)
    float out_scale;            // 1, or the V scale of an fp8 pool: applied where a result is normalised
    float k_inv_scale, v_inv_scale;   // fp8 fused append: 1 / scale of the pools
    int *tickets;               // per (item, kv head): pieces that have arrived; 0 between calls
    // fused append (all NULL for a plain decode call): the item's new K/V row is stored at position len and attended to
    const __nv_bfloat16 *k_new, *v_new;   // [n_items][num_kv_heads][128]
    void *k_pool, *v_pool;                // the pools, writable (bf16 or E4M3 bytes)
    int32_t *seq_lens_out;
    // group decode (NULL otherwise): per item, the first page_offset[i] pages of the table row are skipped
    const int32_t *page_offset;
    float *out_f32;             // when set, result rows go here in fp32 instead of bf16 to `out`
    float *slots;
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
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  The poll has no sleep in it (a sleeping poll wakes up to a microsecond late, which the short
// calls feel).  Gives up when the limit runs out or another warp has already given up; the
// caller carries on (with garbage data) so that every barrier sequence still completes.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, DeviceStatus *status,
                                          int where) {
    if (mbar_try_wait(bar, parity)) return;
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return;
        if ((it & 255u) == 0u) {
            if (*abort_flag) return;
            if (clock64() - t0 > kWaitCycles) break;
        }
    }
    if (*abort_flag == 0) {
        *abort_flag = 1;
        report(status, ROLLART_ERR_TIMEOUT, where, 2);
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
// two bf16 (one 32-bit word) -> two f16
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w) {
    return pack_f16(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
// the two E4M3 bytes in the low (high) half of w -> two f16, low byte first
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2_lo(uint32_t w) {
    uint32_t d;
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tcvt.rn.f16x2.e4m3x2 %0, lo;\n\t}" : "=r"(d) : "r"(w));
    return d;
}
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2_hi(uint32_t w) {
    uint32_t d;
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tcvt.rn.f16x2.e4m3x2 %0, hi;\n\t}" : "=r"(d) : "r"(w));
    return d;
}
// four consecutive result values of one row, at element index idx of the output
__device__ __forceinline__ void store_out4(const DecodeParams &prm, long long idx, float a, float b, float c, float d) {
    if (prm.out_f32 != nullptr) {
        *reinterpret_cast<float4 *>(prm.out_f32 + idx) = make_float4(a, b, c, d);
    } else {
        uint2 packed;
        packed.x = pack_bf16(a, b); packed.y = pack_bf16(c, d);
        *reinterpret_cast<uint2 *>(prm.out + idx) = packed;
    }
}

// One round of the end-of-piece merge: this warp adds (or, in the first round, stores) its two
// 8-dim accumulator tiles of one 16-dim column slice into the shared buffer.
__device__ __forceinline__ void merge_slice(const float (&a)[4], const float (&b)[4], float f0, float f1, float *row0,
                                            float *row1, bool add) {
    float2 a0 = make_float2(a[0] * f0, a[1] * f0), a1 = make_float2(a[2] * f1, a[3] * f1);
    float2 b0 = make_float2(b[0] * f0, b[1] * f0), b1 = make_float2(b[2] * f1, b[3] * f1);
    if (add) {
        const float2 x0 = *reinterpret_cast<float2 *>(row0), x1 = *reinterpret_cast<float2 *>(row1);
        const float2 y0 = *reinterpret_cast<float2 *>(row0 + 8), y1 = *reinterpret_cast<float2 *>(row1 + 8);
        a0.x += x0.x; a0.y += x0.y; a1.x += x1.x; a1.y += x1.y;
        b0.x += y0.x; b0.y += y0.y; b1.x += y1.x; b1.y += y1.y;
    }
    *reinterpret_cast<float2 *>(row0) = a0; *reinterpret_cast<float2 *>(row1) = a1;
    *reinterpret_cast<float2 *>(row0 + 8) = b0; *reinterpret_cast<float2 *>(row1 + 8) = b1;
}

// The same for the fp8 path, whose two accumulator tiles of a 16-dim slice hold, per row, dims 4t, 4t+2 (a) and
// 4t+1, 4t+3 (b) of the slice (t = lane & 3): four consecutive values per row.
__device__ __forceinline__ void merge_slice_fp8(const float (&a)[4], const float (&b)[4], float f0, float f1, float *row0,
                                                float *row1, bool add) {
    float4 x0 = make_float4(a[0] * f0, b[0] * f0, a[1] * f0, b[1] * f0);
    float4 x1 = make_float4(a[2] * f1, b[2] * f1, a[3] * f1, b[3] * f1);
    if (add) {
        const float4 y0 = *reinterpret_cast<float4 *>(row0), y1 = *reinterpret_cast<float4 *>(row1);
        x0.x += y0.x; x0.y += y0.y; x0.z += y0.z; x0.w += y0.w;
        x1.x += y1.x; x1.y += y1.y; x1.z += y1.z; x1.w += y1.w;
    }
    *reinterpret_cast<float4 *>(row0) = x0;
    *reinterpret_cast<float4 *>(row1) = x1;
}

// ------------------------------------------------------------------------------------------
// The walk over a block's span of the tile line: the same code runs in the producer and in the
// consumers, so both see the same sequence of pieces.
// ------------------------------------------------------------------------------------------
struct Piece {
    int item, head, tile0, tile1, ntiles, len;
    int line0;      // where this (item, head) starts on the line
    int advance;    // how far this piece moves the walk along the line
};

// Length of an (item, head) on the line: its tiles plus the fixed cost of a piece.
__device__ __forceinline__ int line_len(int len, int tile_keys) { return len > 0 ? (len + tile_keys - 1) / tile_keys + kPieceCost : 0; }

__device__ __forceinline__ Piece piece_at(const int *prefix, const int *lens, int n_items, int hkv, int p, int p_end) {
    int lo = 0, hi = n_items;                     // largest item with prefix[item] * hkv <= p
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (prefix[mid] * hkv <= p) lo = mid; else hi = mid;
    }
    Piece pc;
    pc.item = lo;
    const int padded = max(1 + kPieceCost, prefix[lo + 1] - prefix[lo]);
    pc.ntiles = padded - kPieceCost;
    const int rem = p - prefix[lo] * hkv;
    pc.head = rem / padded;
    const int off = rem - pc.head * padded;       // position inside the (item, head): tiles first, then the padding
    pc.tile0 = min(off, pc.ntiles);
    pc.tile1 = min(pc.ntiles, off + (p_end - p));
    pc.line0 = p - off;
    pc.advance = min(padded - off, p_end - p);
    pc.len = lens[lo];
    return pc;
}

// ------------------------------------------------------------------------------------------
// Kernel
// ------------------------------------------------------------------------------------------
// kFp8: the pools hold E4M3 bytes (rows of 128 B) instead of bf16 (rows of 256 B).  The schedule, the pieces, the merge
// and the combine are the same; a tile is 128 keys (the same bytes per stage, and half as many hand-overs per byte: a
// warp owns 32 keys of a tile), K and V are converted to f16 as the fragments are loaded and the products run as f16
// MMAs (the query is converted once per piece).
template <bool kFp8>
__global__ void __launch_bounds__(kFp8 ? kThreadsFp8 : kThreads, 1)
decode_splitkv_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap,
                      const DecodeParams prm) {
    constexpr int kS = kStages;                                     // stages of the ring
    constexpr int kSB = kStageBytes;                                // bytes of a stage: K image then V image
    constexpr int kTB = kSB / 2;
    constexpr int kTK = kFp8 ? 2 * kTile : kTile;                   // keys of a tile
    constexpr int kT = kFp8 ? kThreadsFp8 : kThreads;               // threads of the block
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    int *s_lens = reinterpret_cast<int *>(smem + kOffLens);
    int *s_prefix = reinterpret_cast<int *>(smem + kOffPrefix);
    int *s_traj = reinterpret_cast<int *>(smem + kOffTraj);
    float *s_merge = reinterpret_cast<float *>(smem + kOffMerge);
    float *s_ml = reinterpret_cast<float *>(smem + kOffMl);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + kOffAbort);
    const uint32_t bars = smem_u32(smem + kOffBars);
    auto bar_full = [&](int s) { return bars + 8u * s; };
    auto bar_empty = [&](int s) { return bars + 8u * (kS + s); };
    auto bar_qfull = [&](int s) { return bars + 8u * (2 * kS + s); };
    auto bar_qempty = [&](int s) { return bars + 8u * (2 * kS + 2 + s); };
    auto bar_epfull = [&](int s) { return bars + 8u * (2 * kS + 4 + s); };
    auto bar_epempty = [&](int s) { return bars + 8u * (2 * kS + 6 + s); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hkv = prm.num_kv_heads, P = prm.page_size, g = prm.group;

    // Launched with programmatic stream serialisation, this grid may start while the kernel before it in the stream
    // is still draining: let the next launch do the same, set up what needs no global memory, and only then wait
    // for the earlier kernel's results (lengths, pages, tickets) to be complete and visible.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // zero both Q buffers once: rows >= g are never written by the copies and must read as 0
    for (int i = threadIdx.x; i < 2 * kQBytes / 16; i += kT)
        reinterpret_cast<uint4 *>(smem + kOffQ)[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) {
        for (int s = 0; s < kS; ++s) { mbar_init(bar_full(s), 2); mbar_init(bar_empty(s), kConsumerWarps / 2); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar_qfull(s), 1); mbar_init(bar_qempty(s), kConsumerWarps); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar_epfull(s), 1); mbar_init(bar_epempty(s), 1); }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // ---- lengths -> tiles per item -> exclusive prefix (shared memory) ----
    for (int i = threadIdx.x; i < prm.n_items; i += kT) {
        const int t = prm.traj_ids ? __ldg(prm.traj_ids + i) : i + prm.item_offset;
        s_traj[i] = t;
        int L = 0;
        if (t < 0 || t >= prm.num_traj) {
            report(prm.status, ROLLART_ERR_BOUNDS, t, 2);
        } else {
            L = __ldg(prm.seq_lens + t);
            if (prm.k_new != nullptr && L >= 0) {
                // fused append: the new token takes position L; it needs an entry in the page-table row
                if (L / P >= prm.max_pages) { report(prm.status, ROLLART_ERR_BOUNDS, L, 2); L = -1; }
                else L += 1;
            }
            if (L < 0 || L > prm.max_seq_len) { report(prm.status, ROLLART_ERR_BOUNDS, L, 2); L = 0; }
            // the length advances only for an item whose new row is stored (no piece runs for a rejected item)
            if (prm.k_new != nullptr && blockIdx.x == 0 && prm.seq_lens_out != nullptr && L > 0) prm.seq_lens_out[t] = L;
            if (prm.page_offset != nullptr) {
                const int off = __ldg(prm.page_offset + i);
                if (off < 0 || static_cast<long long>(off) * P > L) { report(prm.status, ROLLART_ERR_BOUNDS, off, 2); L = 0; }
                else L -= off * P;
            }
        }
        s_lens[i] = L;
    }
    __syncthreads();
    if (warp == 0) {
        const int per = (prm.n_items + 31) / 32;
        const int a = min(prm.n_items, lane * per), b = min(prm.n_items, a + per);
        int sum = 0;
        for (int i = a; i < b; ++i) sum += line_len(s_lens[i], kTK);
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        int run = incl - sum;
        for (int i = a; i < b; ++i) { s_prefix[i] = run; run += line_len(s_lens[i], kTK); }
        if (lane == 31) s_prefix[prm.n_items] = incl;
    }
    fence_proxy_async();      // the zeroed Q rows are ordered before the bulk copies that land beside them
    __syncthreads();

    if (blockIdx.x == 0) {
        // trajectories without keys have no tile and no piece: their result is out = 0, lse = -inf
        for (int i = 0; i < prm.n_items; ++i) {
            if (s_lens[i] != 0) continue;
            if (prm.out_f32 != nullptr) {
                float4 *o = reinterpret_cast<float4 *>(prm.out_f32 + static_cast<long long>(i) * prm.num_q_heads * kHeadDim);
                for (int k = threadIdx.x; k < prm.num_q_heads * kHeadDim / 4; k += kT) o[k] = make_float4(0.f, 0.f, 0.f, 0.f);
            } else {
                uint4 *o = reinterpret_cast<uint4 *>(prm.out + static_cast<long long>(i) * prm.num_q_heads * kHeadDim);
                for (int k = threadIdx.x; k < prm.num_q_heads * kHeadDim / 8; k += kT) o[k] = make_uint4(0, 0, 0, 0);
            }
            if (prm.lse != nullptr)
                for (int k = threadIdx.x; k < prm.num_q_heads; k += kT)
                    prm.lse[static_cast<long long>(i) * prm.num_q_heads + k] = -INFINITY;
        }
    }
    const int total = s_prefix[prm.n_items] * hkv;
    const int span = max(1, (total + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x));
    const int p_begin = min(total, static_cast<int>(blockIdx.x) * span);
    const int p_end = min(total, p_begin + span);
    if (p_begin >= p_end) return;

    if (warp == kProducerWarp || warp == kProducerWarpV) {
        // =============================== producer warps ===============================
        // Warp 8 brings K (and Q), warp 10 brings V, each with its own arrival on the stage's barrier: a thread is held
        // some 80 cycles by each tensor copy, and with 16-token pages one warp issuing all of them was as slow as the
        // memory (the fp8 pools, with half the bytes per copy, made it the limit).
        const bool do_k = warp == kProducerWarp;
        const int pages_per_tile = kTK / P;
        const int tiles_per_batch = 32 / pages_per_tile;
        const uint32_t page_bytes = static_cast<uint32_t>(P) * (kFp8 ? kHeadDim : kRowBytes);   // one (page, head) image of K or V
        int n = 0, pcount = 0, stage = 0;          // stage = n % kS, phase = (n / kS) & 1, kept as running values
        uint32_t phase = 0;
        bool gave_up = false;
        for (int p = p_begin; p < p_end;) {
            const Piece pc = piece_at(s_prefix, s_lens, prm.n_items, hkv, p, p_end);
            p += pc.advance;
            if (pc.tile0 >= pc.tile1) continue;       // the span touches only the padding of this (item, head)
            const int t = s_traj[pc.item];
            const int32_t *table_row = prm.page_table + static_cast<long long>(t) * prm.max_pages +
                                       (prm.page_offset ? __ldg(prm.page_offset + pc.item) : 0);
            // Q rows of this (item, kv head): g contiguous rows of 256 B
            const int qs = pcount & 1;
            if (do_k) mbar_wait(bar_qempty(qs), ((pcount >> 1) & 1) ^ 1, s_abort, prm.status, 1);
            if (do_k && lane == 0 && !*s_abort) {
                mbar_arrive_expect_tx(bar_qfull(qs), static_cast<uint32_t>(g) * kRowBytes);
                bulk_load(smem_u32(smem + kOffQ + qs * kQBytes),
                          prm.q + (static_cast<long long>(pc.item) * prm.num_q_heads + pc.head * g) * kHeadDim,
                          static_cast<uint32_t>(g) * kRowBytes, bar_qfull(qs));
            }
            // Page ids are fetched 32 at a time, one per lane (8 to 32 tiles' worth), and the next 32 are requested a
            // whole batch ahead, so the table lookup (a dependent load) is off the copy loop's path.
            auto load_ids = [&](int first_tile) {
                const int lp = first_tile * pages_per_tile + lane;
                int pg = -1;
                if (first_tile + lane / pages_per_tile < pc.tile1 && lp * P < pc.len) {
                    pg = __ldg(table_row + lp);
                    if (pg < 0 || pg >= prm.num_pages) { report(prm.status, ROLLART_ERR_BOUNDS, pg, 2); pg = -1; }
                }
                return pg;
            };
            int ids_cur = load_ids(pc.tile0), ids_next = load_ids(pc.tile0 + tiles_per_batch);
            for (int tile = pc.tile0; tile < pc.tile1; ++tile, ++n) {
                const int within = (tile - pc.tile0) & (tiles_per_batch - 1);      // a power of two
                if (tile > pc.tile0 && within == 0) { ids_cur = ids_next; ids_next = load_ids(tile + tiles_per_batch); }
                int pg = __shfl_sync(0xffffffffu, ids_cur, (within * pages_per_tile + lane) & 31);
                if (lane >= pages_per_tile) pg = -1;
                const uint32_t nvalid = __popc(__ballot_sync(0xffffffffu, pg >= 0));
                mbar_wait(bar_empty(stage), phase ^ 1u, s_abort, prm.status, 2);
                if ((n & 15) == 0 && *s_abort) gave_up = true;       // looked at now and then: the copy loop is on the clock
                const int this_stage = stage;
                if (++stage == kS) { stage = 0; phase ^= 1u; }
                if (gave_up) continue;
                if (lane == 0) mbar_arrive_expect_tx(bar_full(this_stage), nvalid * page_bytes);
                __syncwarp();
                if (pg >= 0) {
                    const uint32_t kdst = smem_u32(smem + kOffStages + this_stage * kSB) + lane * page_bytes;
                    const uint32_t vdst = kdst + kTB;
                    const int unit = pg * hkv + pc.head;          // (page, head) tile index
                    if constexpr (kFp8) {
                        // rows of 128 B: one box per (page, head), landing as [slot][128 B]
                        if (do_k) tma_load_2d(kdst, &kmap, bar_full(this_stage), 0, unit * P);
                        else tma_load_2d(vdst, &vmap, bar_full(this_stage), 0, unit * P);
                    } else if (prm.four_d) {
                        if (do_k) tma_load_4d(kdst, &kmap, bar_full(this_stage), 0, 0, 0, unit);
                        else tma_load_4d(vdst, &vmap, bar_full(this_stage), 0, 0, 0, unit);
                    } else {
                        const int row = unit * P;
                        const uint32_t dst = do_k ? kdst : vdst;
                        const CUtensorMap *map = do_k ? &kmap : &vmap;
                        tma_load_2d(dst, map, bar_full(this_stage), 0, row);
                        tma_load_2d(dst + page_bytes / 2, map, bar_full(this_stage), 64, row);
                    }
                }
            }
            ++pcount;
        }
        // every copy this warp issued has been waited for by the consumers unless the block gave up;
        // in that case wait (bounded) for the copies still in flight before the block exits
        if (*s_abort && lane == 0) {
            for (int k = 0; k < kS && k < n; ++k) {
                const int m = n - 1 - k;
                for (uint32_t it = 0; it < kSpinLimit; ++it)
                    if (mbar_try_wait(bar_full(m % kS), (m / kS) & 1)) break;
            }
        }
        return;
    }

    if (warp == kEpilogueWarp) {
        // =============================== epilogue warp ===============================
        // lane -> 4 dims of a row; rows are handled one after the other
        int pcount = 0;
        for (int p = p_begin; p < p_end;) {
            const Piece pc = piece_at(s_prefix, s_lens, prm.n_items, hkv, p, p_end);
            p += pc.advance;
            if (pc.tile0 >= pc.tile1) continue;
            const int eb = pcount & 1;
            mbar_wait(bar_epfull(eb), (pcount >> 1) & 1, s_abort, prm.status, 5);
            const float *mg = s_merge + eb * kMergeFloats;
            const float *ml = s_ml + eb * kMlFloats;
            const bool whole = pc.tile0 == 0 && pc.tile1 == pc.ntiles;
            const int bh = pc.item * hkv + pc.head;
            const long long obase = (static_cast<long long>(pc.item) * prm.num_q_heads + pc.head * g) * kHeadDim + lane * 4;
            const long long lbase = static_cast<long long>(pc.item) * prm.num_q_heads + pc.head * g;
            float *slot = prm.slots + static_cast<size_t>(bh + blockIdx.x) * kSlotFloats;
            // block-level (M, l) of every row: lane r (< 16) owns row r
            float Mrow = -INFINITY, lrow = 0.f;
            if (lane < kMaxGroup) {
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) Mrow = fmaxf(Mrow, ml[(w * kMaxGroup + lane) * 2]);
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    const float mw = ml[(w * kMaxGroup + lane) * 2];
                    if (mw != -INFINITY) lrow += ml[(w * kMaxGroup + lane) * 2 + 1] * exp2f(mw - Mrow);
                }
            }
            if (whole) {
                for (int row = 0; row < g; ++row) {
                    const float lsum = __shfl_sync(0xffffffffu, lrow, row);
                    const float inv = lsum > 0.f ? prm.out_scale / lsum : 0.f;
                    const float4 x = *reinterpret_cast<const float4 *>(mg + row * kMergeStride + lane * 4);
                    store_out4(prm, obase + row * kHeadDim, x.x * inv, x.y * inv, x.z * inv, x.w * inv);
                }
                if (prm.lse != nullptr && lane < g) prm.lse[lbase + lane] = lrow > 0.f ? (Mrow + log2f(lrow)) * kLn2 : -INFINITY;
            } else {
                // Cross-split combine by the last block to arrive.  A block that finds every other piece
                // already published is the last by construction and combines straight from its shared
                // tile; otherwise it publishes its slot (fence, then ticket) and combines only if its
                // ticket turns out to be the last one.  Slots are merged in block order either way.
                // blocks whose spans hold tiles of this (item, head): the padding at its end belongs to no piece
                const int first = pc.line0 / span, last = (pc.line0 + pc.ntiles - 1) / span;
                int arrived = 0;
                if (lane == 0) asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(arrived) : "l"(prm.tickets + bh) : "memory");
                arrived = __shfl_sync(0xffffffffu, arrived, 0);
                int is_last = arrived == last - first;
                if (!is_last) {
                    for (int row = 0; row < g; ++row)
                        *reinterpret_cast<float4 *>(slot + row * kHeadDim + lane * 4) =
                            *reinterpret_cast<const float4 *>(mg + row * kMergeStride + lane * 4);
                    if (lane < g) { slot[kMaxGroup * kHeadDim + lane] = Mrow; slot[kMaxGroup * kHeadDim + kMaxGroup + lane] = lrow; }
                    __threadfence();
                    __syncwarp();
                    if (lane == 0) is_last = atomicAdd(prm.tickets + bh, 1) == last - first;
                    is_last = __shfl_sync(0xffffffffu, is_last, 0);
                }
                if (is_last) {
                    __threadfence();
                    const int row_l = lane < g ? lane : g - 1;          // lanes >= g shadow the last row
                    float Mall = -INFINITY, lall = 0.f;
                    float acc[kMaxGroup][4];
#pragma unroll
                    for (int r = 0; r < kMaxGroup; ++r) acc[r][0] = acc[r][1] = acc[r][2] = acc[r][3] = 0.f;
                    for (int i = first; i <= last; ++i) {
                        const bool mine = i == static_cast<int>(blockIdx.x);
                        const float *sl = prm.slots + static_cast<size_t>(bh + i) * kSlotFloats;
                        float4 x[kMaxGroup];
                        float mi, li;
                        if (mine) {
                            mi = __shfl_sync(0xffffffffu, Mrow, row_l);
                            li = __shfl_sync(0xffffffffu, lrow, row_l);
#pragma unroll
                            for (int r = 0; r < kMaxGroup; ++r)
                                x[r] = *reinterpret_cast<const float4 *>(mg + min(r, g - 1) * kMergeStride + lane * 4);
                        } else {
                            mi = __ldcg(sl + kMaxGroup * kHeadDim + row_l);
                            li = __ldcg(sl + kMaxGroup * kHeadDim + kMaxGroup + row_l);
#pragma unroll
                            for (int r = 0; r < kMaxGroup; ++r)   // all loads issued back to back (rows >= g repeat row g-1)
                                x[r] = __ldcg(reinterpret_cast<const float4 *>(sl + min(r, g - 1) * kHeadDim + lane * 4));
                        }
                        const float Mnew = fmaxf(Mall, mi);
                        const float keep = Mall == -INFINITY ? 0.f : exp2f(Mall - Mnew);
                        const float a_l = mi == -INFINITY ? 0.f : exp2f(mi - Mnew);
                        lall = lall * keep + li * a_l;
                        Mall = Mnew;
#pragma unroll
                        for (int r = 0; r < kMaxGroup; ++r) {
                            const float k = __shfl_sync(0xffffffffu, keep, r), a = __shfl_sync(0xffffffffu, a_l, r);
                            acc[r][0] = acc[r][0] * k + x[r].x * a; acc[r][1] = acc[r][1] * k + x[r].y * a;
                            acc[r][2] = acc[r][2] * k + x[r].z * a; acc[r][3] = acc[r][3] * k + x[r].w * a;
                        }
                    }
#pragma unroll
                    for (int r = 0; r < kMaxGroup; ++r) {
                        const float lsum = __shfl_sync(0xffffffffu, lall, r);
                        if (r < g) {
                            const float inv = lsum > 0.f ? prm.out_scale / lsum : 0.f;
                            store_out4(prm, obase + r * kHeadDim, acc[r][0] * inv, acc[r][1] * inv, acc[r][2] * inv, acc[r][3] * inv);
                        }
                    }
                    if (prm.lse != nullptr && lane < g) prm.lse[lbase + lane] = lall > 0.f ? (Mall + log2f(lall)) * kLn2 : -INFINITY;
                    if (lane == 0) prm.tickets[bh] = 0;                 // every piece has arrived: ready for the next call
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_epempty(eb));      // the shared tile may be refilled
            ++pcount;
        }
        return;
    }

    // ================================= consumer warps =================================
    const int grp = warp >> 2, wq = warp & 3;
    const int qrow = lane >> 2, qcol = lane & 3;          // fragment row / column-pair of this lane
    // byte offset of this warp's 16 keys inside a K (or V) stage image, and ldmatrix lane offsets
    const int key0 = wq * (kFp8 ? 32 : 16);
    // (fp8: the rows of a tile are 128 B and lie one after the other)
    const uint32_t warp_off = kFp8 ? static_cast<uint32_t>(key0 * 128)
                                   : static_cast<uint32_t>((key0 / P) * P * kRowBytes + (key0 % P) * 128);
    const uint32_t half_off = static_cast<uint32_t>(P) * 128;      // second 64 dims of a page image
    const int lm = lane >> 3, lr = lane & 7;
    // K: matrices (keys 0-7 | 8-15) x (dim chunk even | odd)
    const uint32_t k_lane_off = static_cast<uint32_t>(((lm >> 1) * 8 + lr) * 128);
    const int k_chunk_lo = lm & 1;
    // V (transposed load): matrices (keys 0-7 | 8-15) x (dim chunk even | odd of the pair)
    const uint32_t v_lane_off = static_cast<uint32_t>(((lm & 1) * 8 + lr) * 128);
    const int v_chunk_lo = lm >> 1;

    int n = 0, pcount = 0;
    for (int p = p_begin; p < p_end;) {
        const Piece pc = piece_at(s_prefix, s_lens, prm.n_items, hkv, p, p_end);
        p += pc.advance;
        if (pc.tile0 >= pc.tile1) continue;
        const int qs = pcount & 1;
        mbar_wait(bar_qfull(qs), (pcount >> 1) & 1, s_abort, prm.status, 3);
        uint32_t qa[8][4];
        if constexpr (kFp8) {
            // The 16 dims of a step reach the K fragments four bytes per lane (dims 4t .. 4t+3 for t = lane & 3): the
            // step's contraction slots 2t, 2t+1, 2t+8, 2t+9 are those four dims, in the query fragments as well.
            const uint8_t *qrow0 = smem + kOffQ + qs * kQBytes + qrow * kRowBytes + qcol * 8;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint2 lo = *reinterpret_cast<const uint2 *>(qrow0 + ks * 32);
                const uint2 hi = *reinterpret_cast<const uint2 *>(qrow0 + 8 * kRowBytes + ks * 32);
                qa[ks][0] = bf16x2_to_f16x2(lo.x); qa[ks][1] = bf16x2_to_f16x2(hi.x);
                qa[ks][2] = bf16x2_to_f16x2(lo.y); qa[ks][3] = bf16x2_to_f16x2(hi.y);
            }
        } else {
            const uint32_t qbase = smem_u32(smem + kOffQ + qs * kQBytes) + ((lm & 1) * 8 + lr) * kRowBytes + (lm >> 1) * 16;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) ldmatrix_x4(qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], qbase + ks * 32);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_qempty(qs));

        float o[16][4];
#pragma unroll
        for (int j = 0; j < 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

        for (int tile = pc.tile0; tile < pc.tile1; ++tile, ++n) {
            if ((n & 1) != grp) continue;
            const int stage = n % kS;
            mbar_wait(bar_full(stage), (n / kS) & 1, s_abort, prm.status, 4);
            const uint32_t kbase = smem_u32(smem + kOffStages + stage * kSB) + warp_off;
            const uint32_t vbase = kbase + kTB;
            if constexpr (kFp8) {
                // ---- fp8: this warp owns 32 keys of the 128-key tile, as two halves of 16 that share one softmax update ----
                const int valid = min(32, pc.len - tile * kTK - key0);
                bool patched = false;
                if (prm.k_new != nullptr && tile == pc.ntiles - 1 && valid > 0 && pc.len - 1 - tile * kTK - key0 == valid - 1) {
                    // Fused append: this warp owns the context's last key, which is the item's new token.  Its K/V row
                    // comes from k_new / v_new (bf16): it is quantised and put into the staged tile (over whatever the
                    // copy brought for that slot) and into the pool.  Lanes 0-15 move K, lanes 16-31 move V, 8 codes each.
                    const int kk = valid - 1, c8 = lane & 15;
                    const int t = s_traj[pc.item];
                    const int pos = pc.len - 1;
                    const int pg = __ldg(prm.page_table + static_cast<long long>(t) * prm.max_pages + pos / P);
                    const long long src = (static_cast<long long>(pc.item) * hkv + pc.head) * (kHeadDim / 8) + c8;
                    const uint4 val = __ldg(reinterpret_cast<const uint4 *>(lane < 16 ? prm.k_new : prm.v_new) + src);
                    const uint2 code = quantize8(val, lane < 16 ? prm.k_inv_scale : prm.v_inv_scale);
                    const uint32_t a = (lane < 16 ? kbase : vbase) + kk * 128 + (((c8 >> 1) ^ (kk & 7)) << 4) + (c8 & 1) * 8;
                    asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(a), "r"(code.x), "r"(code.y) : "memory");
                    if (pg >= 0 && pg < prm.num_pages) {     // a bad page id was already reported by the producer
                        const long long dst = ((static_cast<long long>(pg) * hkv + pc.head) * P + pos % P) * (kHeadDim / 8) + c8;
                        static_cast<uint2 *>(lane < 16 ? prm.k_pool : prm.v_pool)[dst] = code;
                    }
                    patched = true;
                    __syncwarp();
                }
                if (valid > 0) {
                    if (valid < 32) {
                        // dead slots may hold anything (NaN codes included): zero their V rows so that 0 * v stays 0
                        for (int idx = lane; idx < (32 - valid) * 8; idx += 32) {
                            const uint32_t a = vbase + (valid + (idx >> 3)) * 128 + (idx & 7) * 16;
                            asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0) : "memory");
                        }
                        __syncwarp();
                    }
                    float s[4][4];      // [half * 2 + key octet]
#pragma unroll
                    for (int i = 0; i < 4; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
                    // one load brings keys 0-7 and 8-15 of a half for two 16-dim chunks (a row of 128 B holds 8 chunks of
                    // 16 B); each 32-bit register is the lane's four dims of a key: its halves are the two B registers
#pragma unroll
                    for (int cp = 0; cp < 4; ++cp) {
                        const int chunk = cp * 2 + (lm >> 1);
#pragma unroll
                        for (int hf = 0; hf < 2; ++hf) {
                            uint32_t r0, r1, r2, r3;
                            ldmatrix_x4(r0, r1, r2, r3, kbase + (hf * 16 + (lm & 1) * 8 + lr) * 128 + ((chunk ^ lr) << 4));
                            mma_f16(s[2 * hf], qa[2 * cp], e4m3x2_to_f16x2_lo(r0), e4m3x2_to_f16x2_hi(r0));
                            mma_f16(s[2 * hf + 1], qa[2 * cp], e4m3x2_to_f16x2_lo(r1), e4m3x2_to_f16x2_hi(r1));
                            mma_f16(s[2 * hf], qa[2 * cp + 1], e4m3x2_to_f16x2_lo(r2), e4m3x2_to_f16x2_hi(r2));
                            mma_f16(s[2 * hf + 1], qa[2 * cp + 1], e4m3x2_to_f16x2_lo(r3), e4m3x2_to_f16x2_hi(r3));
                        }
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int col = i * 8 + qcol * 2 + (e & 1);
                            s[i][e] = col < valid ? s[i][e] * prm.scale_log2 : -INFINITY;
                        }
                    float r0 = fmaxf(fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1])), fmaxf(fmaxf(s[2][0], s[2][1]), fmaxf(s[3][0], s[3][1])));
                    float r1 = fmaxf(fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3])), fmaxf(fmaxf(s[2][2], s[2][3]), fmaxf(s[3][2], s[3][3])));
                    r0 = fmaxf(r0, __shfl_xor_sync(0xffffffffu, r0, 1));
                    r0 = fmaxf(r0, __shfl_xor_sync(0xffffffffu, r0, 2));
                    r1 = fmaxf(r1, __shfl_xor_sync(0xffffffffu, r1, 1));
                    r1 = fmaxf(r1, __shfl_xor_sync(0xffffffffu, r1, 2));
                    const float n0 = fmaxf(m0, r0), n1 = fmaxf(m1, r1);
                    if (__any_sync(0xffffffffu, n0 > m0 || n1 > m1)) {
                        const float c0 = exp2f(m0 - n0), c1 = exp2f(m1 - n1);     // exp2(-inf) = 0 on the first tile
                        l0 *= c0; l1 *= c1;
#pragma unroll
                        for (int j = 0; j < 16; ++j) { o[j][0] *= c0; o[j][1] *= c0; o[j][2] *= c1; o[j][3] *= c1; }
                        m0 = n0; m1 = n1;
                    }
                    uint32_t pa[2][4];
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {
                        const float p00 = exp2f(s[2 * hf][0] - m0), p01 = exp2f(s[2 * hf][1] - m0);
                        const float p02 = exp2f(s[2 * hf][2] - m1), p03 = exp2f(s[2 * hf][3] - m1);
                        const float p10 = exp2f(s[2 * hf + 1][0] - m0), p11 = exp2f(s[2 * hf + 1][1] - m0);
                        const float p12 = exp2f(s[2 * hf + 1][2] - m1), p13 = exp2f(s[2 * hf + 1][3] - m1);
                        l0 += (p00 + p01) + (p10 + p11);
                        l1 += (p02 + p03) + (p12 + p13);
                        pa[hf][0] = pack_f16(p00, p01); pa[hf][1] = pack_f16(p02, p03);
                        pa[hf][2] = pack_f16(p10, p11); pa[hf][3] = pack_f16(p12, p13);
                    }
                    // the transposed load hands a lane, for keys 2t and 2t+1, the two dims 2g, 2g+1 of a chunk
                    // (g = lane >> 2): bytes are regrouped into (key 2t, key 2t+1) pairs for the even and the odd
                    // dim, which feed two MMAs; their accumulator columns 2t, 2t+1 are then dims 4t, 4t+2 and
                    // 4t+1, 4t+3 of the chunk
#pragma unroll
                    for (int cp = 0; cp < 4; ++cp) {
                        const int chunk = cp * 2 + (lm >> 1);
#pragma unroll
                        for (int hf = 0; hf < 2; ++hf) {
                            uint32_t r0v, r1v, r2v, r3v;
                            ldmatrix_x4_trans(r0v, r1v, r2v, r3v, vbase + (hf * 16 + (lm & 1) * 8 + lr) * 128 + ((chunk ^ lr) << 4));
                            const uint32_t x0 = __byte_perm(r0v, 0, 0x3120), x1 = __byte_perm(r1v, 0, 0x3120);
                            const uint32_t x2 = __byte_perm(r2v, 0, 0x3120), x3 = __byte_perm(r3v, 0, 0x3120);
                            mma_f16(o[4 * cp], pa[hf], e4m3x2_to_f16x2_lo(x0), e4m3x2_to_f16x2_lo(x1));
                            mma_f16(o[4 * cp + 1], pa[hf], e4m3x2_to_f16x2_hi(x0), e4m3x2_to_f16x2_hi(x1));
                            mma_f16(o[4 * cp + 2], pa[hf], e4m3x2_to_f16x2_lo(x2), e4m3x2_to_f16x2_lo(x3));
                            mma_f16(o[4 * cp + 3], pa[hf], e4m3x2_to_f16x2_hi(x2), e4m3x2_to_f16x2_hi(x3));
                        }
                    }
                    if (valid < 32 || patched) fence_proxy_async();   // our stores into the stage precede the next copy into it
                }
            } else {
                const int valid = min(16, pc.len - tile * kTile - key0);   // live keys among this warp's 16
                bool patched = false;
                if (prm.k_new != nullptr && tile == pc.ntiles - 1 && valid > 0 && valid <= 16 &&
                    pc.len - 1 - tile * kTile - key0 == valid - 1) {
                    // Fused append: this warp owns the context's last key, which is the item's new token.  Its K/V row
                    // comes from k_new / v_new: put it into the staged tile (over whatever the copy brought for that
                    // slot) and into the pool, where later steps will find it.  Lanes 0-15 move K, lanes 16-31 move V.
                    const int kk = valid - 1, c16 = lane & 15;
                    const int t = s_traj[pc.item];
                    const int pos = pc.len - 1;
                    const int pg = __ldg(prm.page_table + static_cast<long long>(t) * prm.max_pages + pos / P);
                    const long long src = (static_cast<long long>(pc.item) * hkv + pc.head) * (kHeadDim / 8) + c16;
                    const uint4 val = __ldg(reinterpret_cast<const uint4 *>(lane < 16 ? prm.k_new : prm.v_new) + src);
                    const uint32_t a = (lane < 16 ? kbase : vbase) + (c16 >> 3) * half_off + kk * 128 + (((c16 & 7) ^ (kk & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(val.x), "r"(val.y), "r"(val.z), "r"(val.w) : "memory");
                    if (pg >= 0 && pg < prm.num_pages) {     // a bad page id was already reported by the producer
                        const long long dst = ((static_cast<long long>(pg) * hkv + pc.head) * P + pos % P) * (kHeadDim / 8) + c16;
                        static_cast<uint4 *>(lane < 16 ? prm.k_pool : prm.v_pool)[dst] = val;
                    }
                    patched = true;
                    __syncwarp();
                }
                if (valid > 0) {
                    if (valid < 16) {
                        // dead slots may hold anything (NaN included): zero their V rows so that 0 * v stays 0
                        for (int idx = lane; idx < (16 - valid) * 16; idx += 32) {
                            const int r = valid + (idx >> 4), c = idx & 15;
                            const uint32_t a = vbase + (c >> 3) * half_off + r * 128 + (c & 7) * 16;
                            asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0) : "memory");
                        }
                        __syncwarp();
                    }
                    float s[2][4];
    #pragma unroll
                    for (int nt = 0; nt < 2; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
    #pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const int chunk = ks * 2 + k_chunk_lo;
                        uint32_t b0, b1, b2, b3;
                        ldmatrix_x4(b0, b1, b2, b3, kbase + (chunk >> 3) * half_off + k_lane_off + (((chunk & 7) ^ lr) << 4));
                        mma_bf16(s[0], qa[ks], b0, b1);
                        mma_bf16(s[1], qa[ks], b2, b3);
                    }
    #pragma unroll
                    for (int nt = 0; nt < 2; ++nt)
    #pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int col = nt * 8 + qcol * 2 + (e & 1);
                            s[nt][e] = col < valid ? s[nt][e] * prm.scale_log2 : -INFINITY;
                        }
                    float r0 = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
                    float r1 = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
                    r0 = fmaxf(r0, __shfl_xor_sync(0xffffffffu, r0, 1));
                    r0 = fmaxf(r0, __shfl_xor_sync(0xffffffffu, r0, 2));
                    r1 = fmaxf(r1, __shfl_xor_sync(0xffffffffu, r1, 1));
                    r1 = fmaxf(r1, __shfl_xor_sync(0xffffffffu, r1, 2));
                    const float n0 = fmaxf(m0, r0), n1 = fmaxf(m1, r1);
                    if (__any_sync(0xffffffffu, n0 > m0 || n1 > m1)) {
                        const float c0 = exp2f(m0 - n0), c1 = exp2f(m1 - n1);     // exp2(-inf) = 0 on the first tile
                        l0 *= c0; l1 *= c1;
    #pragma unroll
                        for (int j = 0; j < 16; ++j) { o[j][0] *= c0; o[j][1] *= c0; o[j][2] *= c1; o[j][3] *= c1; }
                        m0 = n0; m1 = n1;
                    }
                    uint32_t pa[4];
                    {
                        const float p00 = exp2f(s[0][0] - m0), p01 = exp2f(s[0][1] - m0);
                        const float p02 = exp2f(s[0][2] - m1), p03 = exp2f(s[0][3] - m1);
                        const float p10 = exp2f(s[1][0] - m0), p11 = exp2f(s[1][1] - m0);
                        const float p12 = exp2f(s[1][2] - m1), p13 = exp2f(s[1][3] - m1);
                        l0 += (p00 + p01) + (p10 + p11);
                        l1 += (p02 + p03) + (p12 + p13);
                        pa[0] = pack_bf16(p00, p01); pa[1] = pack_bf16(p02, p03);
                        pa[2] = pack_bf16(p10, p11); pa[3] = pack_bf16(p12, p13);
                    }
    #pragma unroll
                    for (int pr = 0; pr < 8; ++pr) {
                        const int chunk = pr * 2 + v_chunk_lo;
                        uint32_t b0, b1, b2, b3;
                        ldmatrix_x4_trans(b0, b1, b2, b3, vbase + (chunk >> 3) * half_off + v_lane_off + (((chunk & 7) ^ lr) << 4));
                        mma_bf16(o[2 * pr], pa, b0, b1);
                        mma_bf16(o[2 * pr + 1], pa, b2, b3);
                    }
                    if (valid < 16 || patched) fence_proxy_async();   // our stores into the stage precede the next copy into it
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty(stage));
        }

        // ---- merge the eight warps into the shared tile of this piece, hand it to the epilogue warp ----
        const int eb = pcount & 1;
        float *mrg = s_merge + eb * kMergeFloats;
        float *ml = s_ml + eb * kMlFloats;
        mbar_wait(bar_epempty(eb), ((pcount >> 1) & 1) ^ 1, s_abort, prm.status, 6);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        if (qcol == 0) {
            ml[(warp * kMaxGroup + qrow) * 2] = m0;       ml[(warp * kMaxGroup + qrow) * 2 + 1] = l0;
            ml[(warp * kMaxGroup + qrow + 8) * 2] = m1;   ml[(warp * kMaxGroup + qrow + 8) * 2 + 1] = l1;
        }
        consumer_bar();
        float M0 = -INFINITY, M1 = -INFINITY;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
            M0 = fmaxf(M0, ml[(w * kMaxGroup + qrow) * 2]);
            M1 = fmaxf(M1, ml[(w * kMaxGroup + qrow + 8) * 2]);
        }
        const float f0 = m0 == -INFINITY ? 0.f : exp2f(m0 - M0);
        const float f1 = m1 == -INFINITY ? 0.f : exp2f(m1 - M1);
#pragma unroll 1
        for (int r = 0; r < kConsumerWarps; ++r) {
            // in round r this warp handles the 16-dim column slice (warp + r) mod 8, so all warps work in
            // every round and each slice receives the warps in a fixed order
            const int c = (warp + r) & 7;
            float *row0 = mrg + qrow * kMergeStride + c * 16 + qcol * (kFp8 ? 4 : 2);
            float *row1 = row0 + 8 * kMergeStride;
            if constexpr (kFp8) {
                switch (c) {
                    case 0: merge_slice_fp8(o[0], o[1], f0, f1, row0, row1, r > 0); break;
                    case 1: merge_slice_fp8(o[2], o[3], f0, f1, row0, row1, r > 0); break;
                    case 2: merge_slice_fp8(o[4], o[5], f0, f1, row0, row1, r > 0); break;
                    case 3: merge_slice_fp8(o[6], o[7], f0, f1, row0, row1, r > 0); break;
                    case 4: merge_slice_fp8(o[8], o[9], f0, f1, row0, row1, r > 0); break;
                    case 5: merge_slice_fp8(o[10], o[11], f0, f1, row0, row1, r > 0); break;
                    case 6: merge_slice_fp8(o[12], o[13], f0, f1, row0, row1, r > 0); break;
                    default: merge_slice_fp8(o[14], o[15], f0, f1, row0, row1, r > 0); break;
                }
            } else
            switch (c) {
                case 0: merge_slice(o[0], o[1], f0, f1, row0, row1, r > 0); break;
                case 1: merge_slice(o[2], o[3], f0, f1, row0, row1, r > 0); break;
                case 2: merge_slice(o[4], o[5], f0, f1, row0, row1, r > 0); break;
                case 3: merge_slice(o[6], o[7], f0, f1, row0, row1, r > 0); break;
                case 4: merge_slice(o[8], o[9], f0, f1, row0, row1, r > 0); break;
                case 5: merge_slice(o[10], o[11], f0, f1, row0, row1, r > 0); break;
                case 6: merge_slice(o[12], o[13], f0, f1, row0, row1, r > 0); break;
                default: merge_slice(o[14], o[15], f0, f1, row0, row1, r > 0); break;
            }
            consumer_bar();
        }
        if (threadIdx.x == 0) mbar_arrive(bar_epfull(eb));
        ++pcount;
    }
}

// ------------------------------------------------------------------------------------------
// Host side: tensor maps
// ------------------------------------------------------------------------------------------
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

bool encode_pool_map(CUtensorMap *map, const void *pool, int num_pages, int hkv, int P, bool four_d) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t units = static_cast<cuuint64_t>(num_pages) * hkv;
    const cuuint32_t ones[4] = {1, 1, 1, 1};
    CUresult r;
    if (four_d) {
        // dims: 64 elements (128 B) | slot | half of the row | (page, head); one box = one (page, head) tile,
        // landing as [half][slot][128 B]
        const cuuint64_t dims[4] = {64, static_cast<cuuint64_t>(P), 2, units};
        const cuuint64_t strides[3] = {kRowBytes, 128, static_cast<cuuint64_t>(P) * kRowBytes};
        const cuuint32_t box[4] = {64, static_cast<cuuint32_t>(P), 2, 1};
        r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(pool), dims, strides, box, ones,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        const cuuint64_t dims[2] = {kHeadDim, units * P};
        const cuuint64_t strides[1] = {kRowBytes};
        const cuuint32_t box[2] = {64, static_cast<cuuint32_t>(P)};
        r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(pool), dims, strides, box, ones,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    return r == CUDA_SUCCESS;
}

// fp8 pool as [rows = pages * heads * slots][128 B]; one box = one (page, head) image of P rows
bool encode_pool_map_fp8(CUtensorMap *map, const void *pool, int num_pages, int hkv, int P) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {kHeadDim, static_cast<cuuint64_t>(num_pages) * hkv * P};
    const cuuint64_t strides[1] = {kHeadDim};
    const cuuint32_t box[2] = {kHeadDim, static_cast<cuuint32_t>(P)};
    const cuuint32_t ones[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(pool), dims, strides, box, ones,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t info_bytes(int items, int hkv) { return (static_cast<size_t>(items) * hkv * sizeof(int2) + 255) & ~size_t(255); }

}  // namespace

size_t decode_workspace_bytes(int max_items, int num_q_heads, int num_kv_heads, int max_seq_len, int sm_count) {
    (void)num_q_heads; (void)max_seq_len; (void)sm_count;
    // per launch (at most kMaxItems items): one ticket counter and one partial slot per
    // (item, kv head), plus one slot per thread block (at most 1024 blocks)
    const int items = max_items < kMaxItems ? max_items : kMaxItems;
    const size_t slots = static_cast<size_t>(items) * num_kv_heads + 1024;
    return info_bytes(items, num_kv_heads) + slots * kSlotFloats * sizeof(float);
}

cudaError_t decode_reset_workspace(void *workspace, size_t bytes, cudaStream_t stream) {
    // the ticket counters sit at the start of the workspace; a kernel that gave up may have left some behind
    const size_t n = bytes < (size_t(1) << 20) ? bytes : (size_t(1) << 20);
    return (workspace != nullptr && n != 0) ? cudaMemsetAsync(workspace, 0, n, stream) : cudaSuccess;
}

cudaError_t launch_decode_attn(const AttnCall &c, cudaStream_t stream, int64_t *launches, bool *too_small) {
    const int hkv = c.pool.num_kv_heads;
    const int chunk_items = c.n_items < kMaxItems ? c.n_items : kMaxItems;
    const size_t need = decode_workspace_bytes(chunk_items, c.num_q_heads, hkv, c.max_seq_len, c.sm_count);
    if (c.workspace == nullptr || need > c.workspace_bytes) { *too_small = true; return cudaErrorInvalidValue; }
    // the tile line of one launch must fit an int
    const long long tiles_bound = ((static_cast<long long>(c.max_seq_len) + kTile - 1) / kTile + kPieceCost) * hkv;
    int per_launch = chunk_items;
    while (per_launch > 1 && tiles_bound * per_launch > 0x3FFFFFFFLL) per_launch /= 2;

    cudaError_t e = cudaFuncSetAttribute(c.fp8 ? decode_splitkv_kernel<true> : decode_splitkv_kernel<false>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    if (c.tma == nullptr) return cudaErrorInvalidValue;
    TmaCache &tc = *c.tma;
    if (!tc.valid || tc.k != c.pool.k || tc.v != c.pool.v || tc.num_pages != c.pool.num_pages || tc.hkv != hkv ||
        tc.page_size != c.pool.page_size || tc.fp8 != (c.fp8 ? 1 : 0)) {
        CUtensorMap *km = reinterpret_cast<CUtensorMap *>(tc.kmap), *vm = reinterpret_cast<CUtensorMap *>(tc.vmap);
        bool four = false;
        if (c.fp8) {
            if (!encode_pool_map_fp8(km, c.pool.k, c.pool.num_pages, hkv, c.pool.page_size) ||
                !encode_pool_map_fp8(vm, c.pool.v, c.pool.num_pages, hkv, c.pool.page_size))
                return cudaErrorInvalidValue;
        } else {
            four = encode_pool_map(km, c.pool.k, c.pool.num_pages, hkv, c.pool.page_size, true) &&
                   encode_pool_map(vm, c.pool.v, c.pool.num_pages, hkv, c.pool.page_size, true);
        }
        if (!four && !c.fp8) {
            if (!encode_pool_map(km, c.pool.k, c.pool.num_pages, hkv, c.pool.page_size, false) ||
                !encode_pool_map(vm, c.pool.v, c.pool.num_pages, hkv, c.pool.page_size, false))
                return cudaErrorInvalidValue;
        }
        tc.four_d = four ? 1 : 0;
        tc.fp8 = c.fp8 ? 1 : 0;
        tc.k = c.pool.k; tc.v = c.pool.v; tc.num_pages = c.pool.num_pages; tc.hkv = hkv; tc.page_size = c.pool.page_size;
        tc.valid = true;
    }

    const int grid = c.sm_count > 0 ? (c.sm_count < 1024 ? c.sm_count : 1024) : 148;
    for (int base = 0; base < c.n_items; base += per_launch) {
        const int n = c.n_items - base < per_launch ? c.n_items - base : per_launch;
        DecodeParams prm;
        prm.page_table = c.trajs.page_table; prm.seq_lens = c.trajs.seq_lens;
        prm.traj_ids = c.traj_ids ? c.traj_ids + base : nullptr;
        prm.max_pages = c.trajs.max_pages; prm.num_traj = c.trajs.num_traj; prm.num_pages = c.pool.num_pages;
        prm.page_size = c.pool.page_size; prm.num_kv_heads = hkv; prm.num_q_heads = c.num_q_heads;
        prm.group = c.num_q_heads / hkv;
        prm.n_items = n; prm.item_offset = base; prm.max_seq_len = c.max_seq_len; prm.four_d = tc.four_d;
        prm.q = c.q + static_cast<long long>(base) * c.num_q_heads * kHeadDim;
        prm.out = c.out + static_cast<long long>(base) * c.num_q_heads * kHeadDim;
        prm.lse = c.lse ? c.lse + static_cast<long long>(base) * c.num_q_heads : nullptr;
        prm.scale_log2 = c.sm_scale * kLog2e * (c.fp8 ? c.k_scale : 1.f);
        prm.out_scale = c.fp8 ? c.v_scale : 1.f;
        prm.k_inv_scale = c.fp8 ? 1.f / c.k_scale : 1.f;
        prm.v_inv_scale = c.fp8 ? 1.f / c.v_scale : 1.f;
        prm.tickets = static_cast<int *>(c.workspace);
        prm.k_new = c.k_new ? c.k_new + static_cast<long long>(base) * hkv * kHeadDim : nullptr;
        prm.v_new = c.v_new ? c.v_new + static_cast<long long>(base) * hkv * kHeadDim : nullptr;
        prm.k_pool = const_cast<__nv_bfloat16 *>(c.pool.k); prm.v_pool = const_cast<__nv_bfloat16 *>(c.pool.v);   // (bytes, for fp8)
        prm.seq_lens_out = c.seq_lens_out;
        prm.page_offset = c.page_offset ? c.page_offset + base : nullptr;
        prm.out_f32 = c.out_f32 ? c.out_f32 + static_cast<long long>(base) * c.num_q_heads * kHeadDim : nullptr;
        prm.slots = reinterpret_cast<float *>(static_cast<char *>(c.workspace) + info_bytes(chunk_items, hkv));
        prm.status = c.status;
        // programmatic stream serialisation: back-to-back decode launches overlap this grid's set-up with the
        // previous grid's tail (the kernel waits for that grid before it reads anything)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid); cfg.blockDim = dim3(c.fp8 ? kThreadsFp8 : kThreads); cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, c.fp8 ? decode_splitkv_kernel<true> : decode_splitkv_kernel<false>,
                               *reinterpret_cast<CUtensorMap *>(tc.kmap), *reinterpret_cast<CUtensorMap *>(tc.vmap), prm);
        ++*launches;
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace rollart

// ==========================================================================================
// Decode attention without any allocation (rollart_decode_attn_noalloc).
//
// The regular entry point keeps its partial slots, ticket counters and status word in memory that
// rollart_create obtained with cudaMalloc.  This variant keeps them in the fixed device array
// below instead, so a caller that must not (or cannot) allocate device memory can still run the
// same kernel.  The array is part of the loaded module: every GPU that loads the library
// holds these bytes until the process exits.
// ==========================================================================================
namespace rollart {
namespace {

constexpr int kStaticMaxUnits = 2048;   // n_items * num_kv_heads per call
constexpr int kStaticMaxGrid = 256;     // thread blocks of the decode kernel in this variant
constexpr size_t kStaticStatusBytes = 256;
constexpr size_t kStaticInfoBytes = static_cast<size_t>(kStaticMaxUnits) * sizeof(int2);
constexpr size_t kStaticSlotBytes = static_cast<size_t>(kStaticMaxUnits + kStaticMaxGrid) * kSlotFloats * sizeof(float);
constexpr size_t kStaticBytes = kStaticStatusBytes + kStaticInfoBytes + kStaticSlotBytes;   // about 19.2 MB

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
struct StaticSetup {
    bool done;
    unsigned char *scratch;   // device address of g_static_scratch on this device
    int sm_count;
};
StaticSetup g_static_setup[kMaxDevices];
std::mutex g_static_mutex;   // guards the per-device set-up

void write_err(char *buf, size_t len, const char *fmt, ...) {
    if (!buf || len == 0) return;
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, len, fmt, ap);
    va_end(ap);
}

}  // namespace
}  // namespace rollart

extern "C" rollart_status rollart_decode_attn_noalloc(int device, const rollart_kv_pool *pool, const rollart_trajs *trajs,
                                                      const int32_t *traj_ids, int32_t n_items, int32_t max_seq_len,
                                                      const void *q, int32_t num_q_heads, float sm_scale, void *out,
                                                      float *lse, int32_t *device_status, void *stream, char *err_buf,
                                                      size_t err_len) {
    using namespace rollart;
    write_err(err_buf, err_len, "ok");
    if (!pool || !trajs || !pool->k_pool || !pool->v_pool || !trajs->page_table || !trajs->seq_lens) {
        write_err(err_buf, err_len, "pool, trajs or one of their pointers is NULL");
        return ROLLART_ERR_INVALID_ARG;
    }
    if (n_items < 0 || max_seq_len < 0 || pool->num_pages <= 0 || pool->num_kv_heads <= 0 || trajs->num_traj <= 0 ||
        trajs->max_pages_per_traj <= 0 || (n_items > 0 && (!q || !out))) {
        write_err(err_buf, err_len, "negative or zero size, or q/out NULL");
        return ROLLART_ERR_INVALID_ARG;
    }
    if (pool->head_dim != kHeadDim || (pool->page_size != 16 && pool->page_size != 32 && pool->page_size != 64)) {
        write_err(err_buf, err_len, "head_dim %d / page_size %d unsupported (128; 16, 32 or 64)", pool->head_dim, pool->page_size);
        return ROLLART_ERR_UNSUPPORTED;
    }
    const int hkv = pool->num_kv_heads;
    if (num_q_heads <= 0 || num_q_heads % hkv != 0) {
        write_err(err_buf, err_len, "num_q_heads %d is not a positive multiple of num_kv_heads %d", num_q_heads, hkv);
        return ROLLART_ERR_INVALID_ARG;
    }
    if (num_q_heads / hkv > kMaxGroup) {
        write_err(err_buf, err_len, "%d query heads per kv head (at most %d)", num_q_heads / hkv, kMaxGroup);
        return ROLLART_ERR_UNSUPPORTED;
    }
    const uintptr_t align_bits = reinterpret_cast<uintptr_t>(pool->k_pool) | reinterpret_cast<uintptr_t>(pool->v_pool) |
                                 reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out);
    if (align_bits & 15u) {
        write_err(err_buf, err_len, "pools, q and out must be 16-byte aligned");
        return ROLLART_ERR_INVALID_ARG;
    }
    // the fixed scratch bounds the call
    if (n_items > kMaxItems || static_cast<long long>(n_items) * hkv > kStaticMaxUnits) {
        write_err(err_buf, err_len,
                  "call too large for the fixed scratch: n_items %d x num_kv_heads %d = %lld (at most %d, and at most %d items)",
                  n_items, hkv, static_cast<long long>(n_items) * hkv, kStaticMaxUnits, kMaxItems);
        return ROLLART_ERR_WORKSPACE;
    }
    const long long cap = static_cast<long long>(trajs->max_pages_per_traj) * pool->page_size;
    if (max_seq_len > cap) max_seq_len = static_cast<int32_t>(cap > 0x7FFFFFFF ? 0x7FFFFFFF : cap);
    if (((static_cast<long long>(max_seq_len) + kTile - 1) / kTile + kPieceCost) * hkv * n_items > 0x3FFFFFFFLL) {
        write_err(err_buf, err_len, "n_items x num_kv_heads x max_seq_len too large for one launch");
        return ROLLART_ERR_WORKSPACE;
    }
    if (device < 0 || device >= kMaxDevices) {
        write_err(err_buf, err_len, "device %d out of range", device);
        return ROLLART_ERR_INVALID_ARG;
    }

    int prev = -1;
    cudaError_t e = cudaGetDevice(&prev);
    if (e == cudaSuccess && prev != device) e = cudaSetDevice(device);
    if (e != cudaSuccess) {
        write_err(err_buf, err_len, "cannot select device %d: %s", device, cudaGetErrorString(e));
        return ROLLART_ERR_CUDA;
    }
    rollart_status result = ROLLART_OK;
    do {
        StaticSetup &su = g_static_setup[device];
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!su.done) {
            // once per device, with that device current: the array's name is only a host-side handle,
            // the kernels need the address it has on this device
            void *ptr = nullptr;
            e = cudaGetSymbolAddress(&ptr, g_static_scratch);
            int major = 0, sms = 0;
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(decode_splitkv_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
            if (e == cudaErrorMemoryAllocation) {
                cudaGetLastError();
                write_err(err_buf, err_len, "set-up on device %d failed: the device has no room left for the library's fixed scratch "
                          "array (%zu bytes, taken when the library's kernels are first loaded): make the first call, which may be "
                          "an empty one, before the device's memory is given away", device, kStaticBytes);
                result = ROLLART_ERR_CUDA;
                break;
            }
            if (e != cudaSuccess || ptr == nullptr) {
                write_err(err_buf, err_len, "set-up on device %d failed: %s", device, cudaGetErrorString(e));
                result = ROLLART_ERR_CUDA;
                break;
            }
            if (major != 10) {
                write_err(err_buf, err_len, "device %d is not an sm_100 GPU", device);
                result = ROLLART_ERR_UNSUPPORTED;
                break;
            }
            su.scratch = static_cast<unsigned char *>(ptr);
            su.sm_count = sms;
            su.done = true;
        }
        if (n_items == 0) break;      // an empty call is the warm-up: the set-up above is all it does
        CUtensorMap kmap, vmap;
        bool four = encode_pool_map(&kmap, pool->k_pool, pool->num_pages, hkv, pool->page_size, true) &&
                    encode_pool_map(&vmap, pool->v_pool, pool->num_pages, hkv, pool->page_size, true);
        if (!four && (!encode_pool_map(&kmap, pool->k_pool, pool->num_pages, hkv, pool->page_size, false) ||
                      !encode_pool_map(&vmap, pool->v_pool, pool->num_pages, hkv, pool->page_size, false))) {
            write_err(err_buf, err_len, "cannot describe the pools to the copy engine (tensor map encode failed)");
            result = ROLLART_ERR_CUDA;
            break;
        }
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        DeviceStatus *status = device_status ? reinterpret_cast<DeviceStatus *>(device_status)
                                             : reinterpret_cast<DeviceStatus *>(su.scratch);
        // the status word and the ticket counters must start at zero (a call that gave up part-way may have
        // left tickets behind); slots are written before they are read
        e = cudaMemsetAsync(su.scratch, 0, kStaticStatusBytes + kStaticInfoBytes, s);
        if (e == cudaSuccess && device_status) e = cudaMemsetAsync(status, 0, sizeof(DeviceStatus), s);
        if (e != cudaSuccess) {
            write_err(err_buf, err_len, "clearing the status word and tickets failed: %s", cudaGetErrorString(e));
            result = ROLLART_ERR_CUDA;
            break;
        }
        DecodeParams prm;
        prm.page_table = trajs->page_table; prm.seq_lens = trajs->seq_lens; prm.traj_ids = traj_ids;
        prm.max_pages = trajs->max_pages_per_traj; prm.num_traj = trajs->num_traj; prm.num_pages = pool->num_pages;
        prm.page_size = pool->page_size; prm.num_kv_heads = hkv; prm.num_q_heads = num_q_heads;
        prm.group = num_q_heads / hkv;
        prm.n_items = n_items; prm.item_offset = 0; prm.max_seq_len = max_seq_len; prm.four_d = four ? 1 : 0;
        prm.q = static_cast<const __nv_bfloat16 *>(q);
        prm.out = static_cast<__nv_bfloat16 *>(out);
        prm.lse = lse;
        prm.scale_log2 = sm_scale * kLog2e;
        prm.out_scale = 1.f;
        prm.k_inv_scale = 1.f; prm.v_inv_scale = 1.f;
        prm.tickets = reinterpret_cast<int *>(su.scratch + kStaticStatusBytes);
        prm.k_new = nullptr; prm.v_new = nullptr; prm.k_pool = nullptr; prm.v_pool = nullptr; prm.seq_lens_out = nullptr;
        prm.page_offset = nullptr; prm.out_f32 = nullptr;
        prm.slots = reinterpret_cast<float *>(su.scratch + kStaticStatusBytes + kStaticInfoBytes);
        prm.status = status;
        const int grid = su.sm_count < kStaticMaxGrid ? su.sm_count : kStaticMaxGrid;
        decode_splitkv_kernel<false><<<grid, kThreads, kSmemBytes, s>>>(kmap, vmap, prm);
        e = cudaGetLastError();
        if (e != cudaSuccess) {
            write_err(err_buf, err_len, "kernel launch failed: %s", cudaGetErrorString(e));
            result = ROLLART_ERR_CUDA;
        }
    } while (false);
    if (prev >= 0 && prev != device) cudaSetDevice(prev);
    return result;
}
