// Chunk attention on the 5th-generation tensor cores (tcgen05 + TMEM), one thread block per unit.
//
// This is the kernel behind the shared-prefix pass of the group decode call (every row of an item sees exactly the
// item's first shared_lens keys, no causal mask, fp32 result + lse); plain causal chunks go to the CTA-pair kernel
// (chunk_attn_pair.cu) through launch_chunk_attn below.  The kernel itself handles both modes.
//
// Work unit: (item, kv head, pair of M-tiles).  An M-tile is 128 query rows = floor(128 / g)
// consecutive chunk tokens x the g query heads that share the kv head, so one K/V read serves all
// of them; a block owns two consecutive M-tiles (256 rows share every K/V tile it brings in) and
// walks the visible keys (the whole cached prefix, then the chunk itself up to the diagonal) in
// tiles of 64 keys.  Per M-tile t and key tile j:
//
//   S_t = Q_t K^T    tcgen05.mma, M 128 x N 64 x K 128, operands in 128B-swizzled shared memory
//                    (Q and K tiles brought by TMA), fp32 accumulator in TMEM, two S buffers per
//                    M-tile so that S(j+1) is computed while the softmax of tile j runs
//   softmax          one warpgroup per M-tile, one thread per query row: tcgen05.ld its 64 scores,
//                    P = exp2(scale * s - m) as packed bf16 stored back with tcgen05.st over the
//                    first 32 columns of the same S buffer, row sum l.  After the first tile m is
//                    not recomputed per tile: the exponentials are taken against the row's current
//                    reference max, and only a row sum that explodes (or a masked tile) sends the
//                    tile down the careful path (row max, new reference, O rescaled in TMEM).  One
//                    pair of exponentials in four is evaluated on the FMA pipe (range reduction +
//                    cubic) to take load off the special-function unit.
//   O_t += P_t V     tcgen05.mma with the A operand (P) in TMEM, M 128 x N 128 x K 64; V is the
//                    MN-major B operand straight from its [key][dim] page layout
//
// Warp roles: warps 0 and 3 issue the copies (0: Q and K, two boxes per page since a QK^T MMA spans the
// keys of several pages; 3: V, one box per page; page ids fetched 32 at a time, a batch ahead), warps 1 and
// 2 each issue the MMAs of one M-tile, warps 4-7 and 8-11 are the two softmax warpgroups, which also
// write the result.  A block uses ~194 KB of shared memory (Q 64 KB, 8 K/V stages of 16 KB) and all
// 512 TMEM columns (2 x 2 S buffers of 64, 2 O accumulators of 128): one block per SM.
// Blocks are ordered (item, kv head, pair), so the blocks that re-read one (item, head)'s keys run
// together and find them in L2.  Every wait is a bounded mbarrier poll; no block waits for another.
#include <cuda.h>

#include <climits>
#include <type_traits>

#include "rollart_internal.cuh"
#include "tc_ptx.cuh"

namespace rollart {

namespace {


constexpr int kRows = 128;                 // query rows of an M-tile (UMMA M)
constexpr int kKeys = 64;                  // keys per KV tile
constexpr int kStages = 8;                 // ring of KV tiles; K(j) and V(j) take alternate slots
constexpr int kThreads = 384;              // warps 0 / 3 copy K / V, warps 1-2 MMA of M-tile 0 / 1, warps 4-7 / 8-11 softmax of M-tile 0 / 1
constexpr int kMaxItems = kChunkItemsPerLaunch;   // items per launch (tile prefix lives in shared memory)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.f;   // log2 units
constexpr float kRowSumLimit = 16777216.f; // 2^24: a tile's row sum above this sends the tile down the careful path
constexpr int kPolyOneIn = 4;              // one pair of exponentials in this many goes to the FMA pipe

constexpr int kHalfQ = kRows * 128;        // 16 KB: 128 rows x 64 dims
constexpr int kTileQ = 2 * kHalfQ;
constexpr int kHalfKV = kKeys * 128;       // 8 KB: 64 keys x 64 dims
constexpr int kTileKV = 2 * kHalfKV;
constexpr int kOffQ = 0;                                   // [M-tile][half][row][128 B]
constexpr int kOffKV = kOffQ + 2 * kTileQ;                 // stages: a K tile is [half][key][128 B], a V tile [page][half][slot][128 B]
constexpr int kOffBars = kOffKV + kStages * kTileKV;
constexpr int kNumBars = 1 + 2 * kStages + 4 + 4 + 4;      // q | kv full/empty | per M-tile and S buffer: s_full, p_full, o_done
constexpr int kOffTmemSlot = kOffBars + kNumBars * 8;
constexpr int kOffAbort = kOffTmemSlot + 8;
constexpr int kOffMl = kOffAbort + 8;                         // (m, l) of the second key stream of a lone M-tile, per row
constexpr int kSmemUsed = kOffMl + kRows * 8;
constexpr int kSmemBytes = kSmemUsed + 1024;               // + slack for the 1024-byte alignment
static_assert(kSmemBytes <= 227 * 1024, "one block must fit an SM");
static_assert((kMaxItems + 1) * 4 <= kStages * kTileKV, "the tile prefix is staged in the KV stages");

constexpr int kTmemCols = 512;             // S buffer b of M-tile t at (2t + b) * 64; O_t at 256 + 128 t; P overwrites the first 32 columns of its S buffer
constexpr int kTmemO = 256;

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
    float out_scale;            // the result is multiplied by this (the value scale of an fp8 cache expanded to bf16; else 1)
    // shared-prefix mode (NULL otherwise): every row of item i sees exactly the first shared_lens[i] keys, no causal mask
    const int32_t *shared_lens;
    float *out_f32;             // when set, result rows go here in fp32 instead of bf16 to `out`
    const int32_t *item_order;  // NULL, or a permutation of the launch's items: blocks take the items in this order
    const uint32_t *redo_bits;  // NULL, or kChunkRedoBits bits: only the units marked there (unit mod kChunkRedoBits) are computed
    DeviceStatus *status;
};

using namespace tc;      // the PTX wrappers and descriptors

// ------------------------------------------------------------------------------------------
// Kernel
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1)
chunk_attn_kernel(const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap kmap,
                  const __grid_constant__ CUtensorMap vmap, const ChunkParams prm) {
    // Second pass behind the CTA-pair kernel: only the units it marked (rows that outgrew their fixed reference max)
    // are computed here, with the same unit numbering; every other block leaves at once.
    if (prm.redo_bits != nullptr) {
        const unsigned u = blockIdx.x;
        if (((__ldg(prm.redo_bits + ((u % kChunkRedoBits) >> 5)) >> (u & 31)) & 1u) == 0u) return;
    }
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hkv = prm.num_kv_heads, P = prm.page_size, g = prm.group;
    const int tpt = kRows / g;                       // chunk tokens per M-tile
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + kOffAbort);
    volatile uint32_t *s_tmem = reinterpret_cast<volatile uint32_t *>(smem + kOffTmemSlot);
    int *s_prefix = reinterpret_cast<int *>(smem + kOffKV);    // staged in the KV stages during the prologue

    if (static_cast<int>(smem - smem_raw) + kSmemUsed > kSmemBytes) {   // cannot happen: the slack covers any alignment
        if (threadIdx.x == 0) report(prm.status, ROLLART_ERR_CUDA, static_cast<int>(smem - smem_raw), 3);
        return;
    }
    const uint32_t bars = smem_u32(smem + kOffBars);
    const uint32_t bar_q = bars;
    // ring slot r (K(j) is r = 2j, V(j) is r = 2j + 1) lives in stage r % kStages
    auto bar_full = [&](int s) { return bars + 8u * (1 + s); };
    auto bar_empty = [&](int s) { return bars + 8u * (1 + kStages + s); };
    // key tile j of M-tile t uses S buffer b = j & 1 and the barriers of (t, b): a warp that is a tile ahead of the
    // others of its warpgroup arrives on the other barrier
    auto bar_sfull = [&](int t, int b) { return bars + 8u * (1 + 2 * kStages + 2 * t + b); };
    auto bar_pfull = [&](int t, int b) { return bars + 8u * (1 + 2 * kStages + 4 + 2 * t + b); };
    auto bar_odone = [&](int t, int b) { return bars + 8u * (1 + 2 * kStages + 8 + 2 * t + b); };

    // ---- which (item, kv head, pair of M-tiles) is this block?  pairs per item -> prefix -> search ----
    auto ordered = [&](int k) {        // the k-th item to be taken (clamped: the order is only a schedule, never an index check)
        if (prm.item_order == nullptr) return k;
        return min(max(__ldg(prm.item_order + k), 0), prm.n_items - 1);
    };
    for (int i = threadIdx.x; i < prm.n_items; i += kThreads) {
        const int it = ordered(i);
        const int n = __ldg(prm.q_indptr + it + 1) - __ldg(prm.q_indptr + it);
        s_prefix[i + 1] = n > 0 ? (n + 2 * tpt - 1) / (2 * tpt) : 0;
    }
    if (threadIdx.x == 0) {
        s_prefix[0] = 0;
        mbar_init(bar_q, 1);
        for (int s = 0; s < kStages; ++s) mbar_init(bar_full(s), 1);      // the empty barriers count the live M-tiles: set up below
        for (int t = 0; t < 2; ++t)
            for (int b = 0; b < 2; ++b) { mbar_init(bar_sfull(t, b), 1); mbar_init(bar_odone(t, b), 1); mbar_init(bar_pfull(t, b), 4); }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (warp == 0) {        // inclusive scan of the pair counts, in place
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
    int item = 0, head = 0, pair = 0;
    if (unit < total_units) {
        int lo = 0, hi = prm.n_items;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_prefix[mid] * hkv <= unit) lo = mid; else hi = mid;
        }
        item = ordered(lo);
        const int np = max(1, s_prefix[lo + 1] - s_prefix[lo]);
        const int rem = unit - s_prefix[lo] * hkv;
        head = rem / np;
        pair = np - 1 - (rem - head * np);      // later M-tiles see more keys: start the longest ones first
    }
    __syncthreads();                 // everyone has read the prefix: the KV stages are free again
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
    const int tok0 = pair * 2 * tpt;                            // first chunk token of M-tile 0
    // per M-tile: live tokens, keys visible to its last live row / first row, key tiles (M-tile 1 may be absent)
    int toks_[2], maxc_[2], minc_[2], nt_[2];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
        const int first = tok0 + mt * tpt;
        toks_[mt] = max(0, min(tpt, n_chunk - first));
        maxc_[mt] = toks_[mt] == 0 ? 0 : (shared_mode ? L : prior + first + toks_[mt]);
        minc_[mt] = shared_mode ? L : prior + first + 1;
        nt_[mt] = (maxc_[mt] + kKeys - 1) / kKeys;
    }
    const int n0 = nt_[0], n1 = nt_[1], nmax = max(n0, n1);
    // A lone M-tile (the ragged end of a chunk, or a small shared-prefix group) would leave half of the block idle:
    // its key tiles are then dealt alternately to the two halves (even tiles to MMA thread / warpgroup 0, odd tiles
    // to 1), each with its own S buffers, running max, sum and O accumulator, and the two are merged at the end.
    const bool split = n1 == 0 && n0 >= 2;
    const int step = split ? 2 : 1;
    const int32_t *table_row = prm.page_table + static_cast<long long>(t) * prm.max_pages;
    if (nmax == 0) {
        // only in shared-prefix mode with an empty prefix: the result is out = 0, lse = -inf
        const int toks = toks_[0] + toks_[1];
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

    // zero the Q tiles (rows beyond tpt * g are never written by the copy) and allocate TMEM
    for (int i = threadIdx.x; i < 2 * kTileQ / 16; i += kThreads) reinterpret_cast<uint4 *>(smem + kOffQ)[i] = make_uint4(0, 0, 0, 0);
    fence_proxy_async();
    if (threadIdx.x == 32) {
        for (int s = 0; s < kStages; ++s) mbar_init(bar_empty(s), n1 > 0 ? 2 : 1);     // readers of a K/V tile
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc(smem_u32(smem + kOffTmemSlot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *s_tmem;

    if (warp == 0 || warp == 3) {
        // =============================== copy warps ===============================
        // Warp 0 brings the Q tiles and every K tile, warp 3 every V tile: a thread is held for some 80 cycles by each
        // tensor copy it issues, and twelve of them per key tile from one warp were close to the tile period.
        const int kv = warp == 3 ? 1 : 0;
        if (kv == 0 && lane == 0) {
            const int live_tiles = n1 > 0 ? 2 : 1;
            mbar_arrive_expect_tx(bar_q, static_cast<uint32_t>(live_tiles * tpt * g) * kRowBytes);
            for (int mt = 0; mt < live_tiles; ++mt) {
                const uint32_t dst = smem_u32(smem + kOffQ + mt * kTileQ);
                tma_load_3d(dst, &qmap, bar_q, 0, head * g, q_row0 + tok0 + mt * tpt);
                tma_load_3d(dst + kHalfQ, &qmap, bar_q, 64, head * g, q_row0 + tok0 + mt * tpt);
            }
        }
        const int pages_per_tile = kKeys / P;
        const int tiles_per_batch = 32 / pages_per_tile;
        const uint32_t half_page = static_cast<uint32_t>(P) * 128;
        // Page ids are fetched 32 at a time, one per lane (enough for 8 to 32 key tiles), and the next 32 are
        // requested a whole batch ahead, so the table lookup (a dependent load) is off the copy loop's path.
        auto load_ids = [&](int batch) {
            const int lp = batch * 32 + lane;
            int pg = -1;
            if (lp * P < L && lp < prm.max_pages) {
                pg = __ldg(table_row + lp);
                if (pg < 0 || pg >= prm.num_pages) {
                    if (kv == 0) report(prm.status, ROLLART_ERR_BOUNDS, pg, 3);
                    pg = -1;
                }
            }
            return pg;
        };
        int ids_cur = load_ids(0), ids_next = load_ids(1);
        for (int j = 0; j < nmax; ++j) {
            const int within = j % tiles_per_batch;
            if (j > 0 && within == 0) {
                if (*s_abort) break;
                ids_cur = ids_next;
                ids_next = load_ids(j / tiles_per_batch + 1);
            }
            int pg = __shfl_sync(0xffffffffu, ids_cur, (within * pages_per_tile + lane) & 31);
            if (lane >= pages_per_tile) pg = -1;
            const uint32_t nvalid = __popc(__ballot_sync(0xffffffffu, pg >= 0));
            const int r = 2 * j + kv, stage = r % kStages;       // K(j) and V(j) take alternate slots of the ring
            mbar_wait(bar_empty(stage), ((r / kStages) & 1) ^ 1, s_abort, prm.status, 1 + kv);
            if (lane == 0) mbar_arrive_expect_tx(bar_full(stage), nvalid * 2u * half_page);
            __syncwarp();
            if (pg >= 0) {
                const uint32_t stage_addr = smem_u32(smem + kOffKV + stage * kTileKV);
                if (kv == 0) {
                    // K tile as [half][key][128 B]: two boxes per page (a QK^T MMA spans the keys of all pages)
                    const int row = (pg * hkv + head) * P;
                    tma_load_2d(stage_addr + lane * half_page, &kmap, bar_full(stage), 0, row);
                    tma_load_2d(stage_addr + lane * half_page + kHalfKV, &kmap, bar_full(stage), 64, row);
                } else {
                    // V tile as [page][half][slot][128 B]: one box per page (a PV MMA step stays inside a page)
                    tma_load_4d(stage_addr + lane * 2u * half_page, &vmap, bar_full(stage), 0, 0, 0, pg * hkv + head);
                }
            }
        }
    } else if (warp == 1 || warp == 2) {
        // =============================== MMA warps ===============================
        // One issuing thread per M-tile: warp 1 runs QK_0 / PV_0, warp 2 runs QK_1 / PV_1.  A thread that issues an
        // MMA is held until the tensor core accepts it, so everything else that thread does between two MMAs is time
        // the tensor core may idle; with one thread per M-tile each has half the MMAs and the waits of one M-tile do
        // not delay the other's products.  Per thread the order is QK(0) | QK(j+1) PV(j) | ...: S of the next key
        // tile is ready before the softmax of this one ends.  MMAs of one thread run in issue order, which is what
        // protects the reuse of an S buffer (it holds P(j-1) until PV(j-1), issued before QK(j+1), has read it).
        // Both threads release every KV stage (its barrier counts the live M-tiles), also for key tiles their own
        // M-tile does not use.
        const int mt = warp - 1;
        // key tiles of this thread: j = first + i * step for i < cnt
        const int first = split ? mt : 0;
        const int cnt = split ? (n0 - mt + 1) / 2 : (mt == 0 ? n0 : n1);
        if (lane == 0 && cnt > 0) {
            constexpr uint32_t kIdescQK = idesc(kRows, kKeys, false);
            constexpr uint32_t kIdescPV = idesc(kRows, kHeadDim, true);
            const uint32_t kv_addr = smem_u32(smem + kOffKV);
            const uint64_t q_desc = smem_desc(smem_u32(smem + kOffQ) + (split ? 0 : mt) * kTileQ, 16);
            const uint32_t s_tmem = tmem + mt * 2 * kKeys, o_tmem = tmem + kTmemO + mt * kHeadDim;
            // V stage image is [page][half][slot][128 B]: the 16 keys of PV step ks sit in page (16 ks) / P at slot
            // (16 ks) % P; the two 64-dim halves of a page are P * 128 B apart
            const uint32_t v_half = static_cast<uint32_t>(P) * 128u;
            uint64_t v_off[kKeys / 16];
#pragma unroll
            for (int ks = 0; ks < kKeys / 16; ++ks)
                v_off[ks] = static_cast<uint64_t>((((ks * 16) / P) * P * kRowBytes + ((ks * 16) % P) * 128) >> 4);
            auto full_wait = [&](int r, int where) {
                mbar_wait(bar_full(r % kStages), (r / kStages) & 1, s_abort, prm.status, where);
            };
            auto issue_qk = [&](int i) {
                const int j = first + i * step;
                full_wait(2 * j, 6);                        // K(j)
                tc_fence_after();
                const uint64_t k_desc = smem_desc(kv_addr + ((2 * j) % kStages) * kTileKV, 16);
#pragma unroll
                for (int ks = 0; ks < kHeadDim / 16; ++ks) {   // 16 dims per step; the second 64 dims live in the other half
                    const uint64_t qoff = static_cast<uint64_t>(((ks >> 2) * kHalfQ + (ks & 3) * 32) >> 4);
                    const uint64_t koff = static_cast<uint64_t>(((ks >> 2) * kHalfKV + (ks & 3) * 32) >> 4);
                    umma_bf16(s_tmem + (i & 1) * kKeys, q_desc + qoff, k_desc + koff, kIdescQK, ks > 0 ? 1u : 0u);
                }
                umma_commit(bar_sfull(mt, i & 1));
                umma_commit(bar_empty((2 * j) % kStages));
            };
            mbar_wait(bar_q, 0, s_abort, prm.status, 5);
            issue_qk(0);
            for (int i = 0; i < cnt; ++i) {
                const int j = first + i * step;
                if (i + 1 < cnt) issue_qk(i + 1);
                full_wait(2 * j + 1, 3);                    // V(j)
                mbar_wait(bar_pfull(mt, i & 1), (i >> 1) & 1, s_abort, prm.status, 4);
                tc_fence_after();
                const uint64_t v_desc = smem_desc(kv_addr + ((2 * j + 1) % kStages) * kTileKV, v_half);
                const uint32_t acc0 = i > 0 ? 1u : 0u;
#pragma unroll
                for (int ks = 0; ks < kKeys / 16; ++ks)     // 16 keys per step: 8 packed columns along P's row
                    umma_bf16_ts(o_tmem, s_tmem + (i & 1) * kKeys + ks * 8, v_desc + v_off[ks], kIdescPV, ks > 0 ? 1u : acc0);
                umma_commit(bar_odone(mt, i & 1));
                umma_commit(bar_empty((2 * j + 1) % kStages));   // V(j)
            }
            // key tiles that only the other M-tile uses (it sees more keys): this thread releases them unread
            if (!split)
                for (int j = cnt; j < nmax; ++j) {
                    full_wait(2 * j, 6);
                    umma_commit(bar_empty((2 * j) % kStages));
                    full_wait(2 * j + 1, 3);
                    umma_commit(bar_empty((2 * j + 1) % kStages));
                }
        }
        __syncwarp();
    } else if (warp >= 4) {
        // =============================== softmax warpgroups ===============================
        const int mt = (warp - 4) >> 2;                       // M-tile of this warpgroup
        const int wg_thread = ((warp - 4) & 3) * 32 + lane;
        const int quarter = warp & 3;                         // TMEM lanes 32 * quarter .. + 31 belong to this warp
        const int row = quarter * 32 + lane;
        const uint32_t lane_addr = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        const uint32_t s_addr = lane_addr + mt * 2 * kKeys, o_addr = lane_addr + kTmemO + mt * kHeadDim;
        // key tiles of this warpgroup: j = first + i * step for i < cnt; a lone M-tile (split) is M-tile 0 for both
        const int first = split ? mt : 0;
        const int cnt = split ? (n0 - mt + 1) / 2 : (mt == 0 ? n0 : n1);
        const int gt = split ? 0 : mt;                         // whose rows these are
        const int toks = gt == 0 ? toks_[0] : toks_[1];
        const int min_count = gt == 0 ? minc_[0] : minc_[1];
        const int first_tok = tok0 + gt * tpt;
        const int tok_local = row / g, head_local = row - tok_local * g;
        const bool live = tok_local < toks;
        const int count = shared_mode ? L : min(L, prior + first_tok + min(tok_local, max(toks, 1) - 1) + 1);   // keys this row sees (>= 1)
        const float scale = prm.scale_log2;
        float m_ref = -INFINITY, l_sum = 0.f;

        for (int i = 0; i < cnt; ++i) {
            const int j = first + i * step;
            const int sb = i & 1;
            const uint32_t sbuf = s_addr + sb * kKeys;
            mbar_wait(bar_sfull(mt, sb), (i >> 1) & 1, s_abort, prm.status, 8);
            tc_fence_after();
            uint32_t sraw[2][32];
            tmem_ld32(sbuf, sraw[0]);
            tmem_ld32(sbuf + 32, sraw[1]);
            tmem_wait_ld();

            const int key0 = j * kKeys;
            const bool need_mask = key0 + kKeys > min_count;    // uniform over the warpgroup
            const int live_keys = count - key0;                 // keys of this tile the row sees (masked tiles only)
            float rs[4];
            // two copies of the pass, chosen once per tile: the unmasked one (every tile but the last few of an
            // M-tile) carries no compare / select per element
            int poly_top = INT_MIN;     // the largest argument handed to the FMA-pipe exponential (see ex2_poly2)
            auto exp_pass = [&](auto masked_tag, auto poly_tag, float neg_m) {
                constexpr bool kMasked = decltype(masked_tag)::value;
                constexpr bool kPoly = decltype(poly_tag)::value;
                rs[0] = rs[1] = rs[2] = rs[3] = 0.f;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t packed[16];
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        float x0, x1, p0, p1;
                        fma2(x0, x1, __uint_as_float(sraw[h][c]), __uint_as_float(sraw[h][c + 1]), scale, neg_m);
                        if (kPoly && ((c >> 1) % kPolyOneIn) == kPolyOneIn - 1) {
                            ex2_poly2(p0, p1, x0, x1, poly_top);
                        } else {
                            p0 = ex2(x0);
                            p1 = ex2(x1);
                        }
                        if constexpr (kMasked) {
                            p0 = h * 32 + c < live_keys ? p0 : 0.f;
                            p1 = h * 32 + c + 1 < live_keys ? p1 : 0.f;
                        }
                        add2(rs[c & 2], rs[(c & 2) + 1], p0, p1);
                        packed[c >> 1] = pack_bf16(p0, p1);
                    }
                    // P as the next A operand: 64 bf16 of this row as 32 packed columns over the start of its S buffer
                    tmem_st16(sbuf + h * 16, packed);
                }
                return (rs[0] + rs[1]) + (rs[2] + rs[3]);
            };
            // Fast path (every unmasked tile after the first): no max pass.  The exponentials are taken against the
            // row's current reference max m_ref, which is the max of some earlier score, so later keys far below it
            // rightly vanish; keys far above it make the row sum explode, and then (rarely) the tile is redone the
            // careful way below.  Up to that bound P and the sums just carry a larger exponent: fp32 accumulation
            // and the 8-bit mantissa of bf16 P lose nothing by it.
            float rsum = 0.f, corr = 1.f;
            bool careful = i == 0 || need_mask;
            if (!careful) {
                rsum = exp_pass(std::false_type{}, std::true_type{}, -m_ref);
                // also true for inf / NaN, and for a score so far above the reference that the FMA-pipe exponential broke
                careful = __any_sync(0xffffffffu, !(rsum <= kRowSumLimit) || poly_top > kPolyArgTop);
                if (careful) tmem_wait_st();      // the stores of the abandoned pass land before the new ones
            }
            if (careful) {
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
                    // masked tile: keys the row does not see are left out (their scores may be anything)
                    rmax = -INFINITY;
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (h * 32 + c < live_keys) rmax = fmaxf(rmax, __uint_as_float(sraw[h][c]) * scale);
                }
                // the reference max moves only when it has to (first tile) or when a row outgrew it by 2^8
                const bool grow = rmax > m_ref + kRescaleThreshold;
                const float m_new = grow ? rmax : m_ref;
                corr = grow ? ex2(m_ref - m_new) : 1.f;   // ex2(-inf) = 0 on the first tile
                if (i >= 1 && __any_sync(0xffffffffu, grow)) {
                    // rare: some row of this warp moved its reference max, so O (the tiles before this one) must be
                    // rescaled before PV of this tile; PV of the previous tile has to be finished first
                    mbar_wait(bar_odone(mt, (i - 1) & 1), ((i - 1) >> 1) & 1, s_abort, prm.status, 9);
                    tc_fence_after();
#pragma unroll 1
                    for (int c0 = 0; c0 < kHeadDim; c0 += 16) {
                        uint32_t oraw[16];
                        tmem_ld16(o_addr + c0, oraw);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 16; ++c) oraw[c] = __float_as_uint(__uint_as_float(oraw[c]) * corr);
                        tmem_st16(o_addr + c0, oraw);
                    }
                }
                m_ref = m_new;
                // (every exponential on the special-function unit here: the careful path has no bound on its arguments to rely on)
                rsum = need_mask ? exp_pass(std::true_type{}, std::false_type{}, -m_ref)
                                 : exp_pass(std::false_type{}, std::false_type{}, -m_ref);
            }
            l_sum = l_sum * corr + rsum;
            tmem_wait_st();
            if (key0 + kKeys > L) {
                // keys at or beyond L are dead slots (or were never copied): their V rows must be 0, not garbage.
                // Each warpgroup does it before releasing its own PV (the two may both write the same zeros).
                const int r = 2 * j + 1;
                mbar_wait(bar_full(r % kStages), (r / kStages) & 1, s_abort, prm.status, 10);
                const uint32_t v_addr = smem_u32(smem + kOffKV + (r % kStages) * kTileKV);
                const int first_dead = L - key0;
                for (int idx = wg_thread; idx < (kKeys - first_dead) * 16; idx += 128) {
                    const int rr = first_dead + (idx >> 4), c = idx & 15;
                    const uint32_t a = v_addr + (rr / P) * (P * kRowBytes) + (c >> 3) * (P * 128) + (rr % P) * 128 + (c & 7) * 16;
                    asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0) : "memory");
                }
                fence_proxy_async();      // the zeroed V rows become visible to the tensor core's reads
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_pfull(mt, sb));
        }

        // ---- epilogue: O / l -> bf16 rows of out ----
        if (cnt > 0) {
            mbar_wait(bar_odone(mt, (cnt - 1) & 1), ((cnt - 1) >> 1) & 1, s_abort, prm.status, 11);
            tc_fence_after();
        }
        float w0 = 1.f, w1 = 0.f;                // weights of the two key streams of a lone M-tile
        if (split) {
            // warpgroup 1 hands its (m, l) to warpgroup 0, which owns the same TMEM lanes and reads both accumulators
            float *ml = reinterpret_cast<float *>(smem + kOffMl);
            if (mt == 1) { ml[2 * row] = m_ref; ml[2 * row + 1] = l_sum; }
            tc_fence_before();
            asm volatile("bar.sync 1, 256;" ::: "memory");
            tc_fence_after();
            if (mt == 0) {
                const float m1 = ml[2 * row], l1 = ml[2 * row + 1];
                const float m_all = fmaxf(m_ref, m1);
                w0 = m_ref == -INFINITY ? 0.f : ex2(m_ref - m_all);
                w1 = m1 == -INFINITY ? 0.f : ex2(m1 - m_all);
                l_sum = l_sum * w0 + l1 * w1;
                m_ref = m_all;
            }
        }
        if (cnt > 0 && !(split && mt == 1)) {
            const float inv = l_sum > 0.f ? prm.out_scale / l_sum : 0.f;
            const float f0 = w0 * inv, f1 = w1 * inv;
            const long long orow = (static_cast<long long>(q_row0 + first_tok + tok_local) * prm.num_q_heads + head * g + head_local);
#pragma unroll 1
            for (int c0 = 0; c0 < kHeadDim; c0 += 32) {
                uint32_t oraw[32];
                tmem_ld32(o_addr + c0, oraw);
                tmem_wait_ld();
                float ov[32];
#pragma unroll
                for (int k = 0; k < 32; ++k) ov[k] = __uint_as_float(oraw[k]) * f0;
                if (split) {                     // uniform over the block
                    tmem_ld32(o_addr + kHeadDim + c0, oraw);
                    tmem_wait_ld();
#pragma unroll
                    for (int k = 0; k < 32; ++k) ov[k] = fmaf(__uint_as_float(oraw[k]), f1, ov[k]);
                }
                if (live && prm.out_f32 != nullptr) {
                    float4 *dst = reinterpret_cast<float4 *>(prm.out_f32 + orow * kHeadDim + c0);
#pragma unroll
                    for (int k = 0; k < 8; ++k) dst[k] = make_float4(ov[4 * k], ov[4 * k + 1], ov[4 * k + 2], ov[4 * k + 3]);
                } else if (live) {
                    uint4 *dst = reinterpret_cast<uint4 *>(prm.out + orow * kHeadDim + c0);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        uint4 v;
                        v.x = pack_bf16(ov[8 * k], ov[8 * k + 1]);
                        v.y = pack_bf16(ov[8 * k + 2], ov[8 * k + 3]);
                        v.z = pack_bf16(ov[8 * k + 4], ov[8 * k + 5]);
                        v.w = pack_bf16(ov[8 * k + 6], ov[8 * k + 7]);
                        dst[k] = v;
                    }
                }
            }
            if (live && prm.lse != nullptr) prm.lse[orow] = l_sum > 0.f ? (m_ref + log2f(l_sum)) * kLn2 : -INFINITY;
        }
        tc_fence_before();
    }

    // ---- all roles meet; the allocating warp returns the TMEM columns ----
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// Diagnostic: one thread waits, with the bounded wait every role of the tensor-core kernels uses, on a barrier that
// nothing arrives at.  The wait gives up when its limit (about a second) runs out and records ROLLART_ERR_TIMEOUT.
__global__ void bounded_wait_selftest_kernel(DeviceStatus *status) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(smem_u32(&bar), 0, &abort_flag, status, 15);
    }
}

}  // namespace

cudaError_t launch_chunk_attn(const AttnCall &c, cudaStream_t stream, int64_t *launches, bool *too_small) {
    (void)too_small;
    // Plain causal chunks run on CTA pairs (chunk_attn_pair.cu), whose rows keep the reference max of their first key
    // tile; the units in which a row outgrew it are marked in a bitmap and computed again here, by the kernel that
    // moves its reference max (a launch whose other blocks leave at once).  This kernel also keeps the shared-prefix
    // mode of the group decode call (one M-tile per group: a pair would idle its second CTA, and that pass is bound by
    // memory).
    const bool plain = c.shared_lens == nullptr && c.out_f32 == nullptr && c.item_order == nullptr;
    if (plain && c.redo_bits == nullptr) return cudaErrorInvalidValue;
    const int hkv = c.pool.num_kv_heads, g = c.num_q_heads / hkv, tpt = kRows / g;
    cudaError_t e = cudaFuncSetAttribute(chunk_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    CUtensorMap qmap, kmap, vmap;
    if (!encode_q_map(&qmap, c.q, c.total_q, c.num_q_heads, g) ||
        !encode_pool_rows(&kmap, c.pool.k, c.pool.num_pages, hkv, c.pool.page_size) ||
        !encode_pool_pages(&vmap, c.pool.v, c.pool.num_pages, hkv, c.pool.page_size))
        return cudaErrorInvalidValue;
    for (int base = 0; base < c.n_items; base += kMaxItems) {
        const int n = c.n_items - base < kMaxItems ? c.n_items - base : kMaxItems;
        if (plain) {
            e = cudaMemsetAsync(c.redo_bits, 0, kChunkRedoBits / 8 + 64, stream);      // the bitmap and, behind it, the pair kernel's unit counter
            if (e != cudaSuccess) return e;
            e = launch_chunk_attn_pair(c, base, n, stream, launches);
            if (e != cudaSuccess) return e;
        }
        ChunkParams prm;
        prm.page_table = c.trajs.page_table; prm.seq_lens = c.trajs.seq_lens;
        prm.traj_ids = c.traj_ids ? c.traj_ids + base : nullptr;
        prm.q_indptr = c.q_indptr + base;
        prm.max_pages = c.trajs.max_pages; prm.num_traj = c.trajs.num_traj; prm.num_pages = c.pool.num_pages;
        prm.page_size = c.pool.page_size; prm.num_kv_heads = hkv; prm.num_q_heads = c.num_q_heads; prm.group = g;
        prm.n_items = n; prm.item_offset = base; prm.max_seq_len = c.max_seq_len; prm.total_q = c.total_q;
        prm.out = c.out; prm.lse = c.lse; prm.scale_log2 = c.sm_scale * kLog2e; prm.out_scale = c.v_scale; prm.status = c.status;
        prm.shared_lens = c.shared_lens ? c.shared_lens + base : nullptr;
        prm.out_f32 = c.out_f32;
        prm.item_order = c.item_order ? c.item_order + base : nullptr;
        prm.redo_bits = plain ? c.redo_bits : nullptr;
        // an upper bound on the M-tile pairs of these items: every item has at most one ragged pair
        const long long pairs = (static_cast<long long>(c.total_q) + 2 * tpt - 1) / (2 * tpt) + n;
        const long long blocks = pairs * hkv;
        if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
        chunk_attn_kernel<<<static_cast<unsigned>(blocks), kThreads, kSmemBytes, stream>>>(qmap, kmap, vmap, prm);
        ++*launches;
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_bounded_wait_selftest(DeviceStatus *status, cudaStream_t stream, int64_t *launches) {
    bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(status);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace rollart
