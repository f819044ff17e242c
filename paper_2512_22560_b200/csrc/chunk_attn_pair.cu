// Observation-chunk attention on CTA pairs: two thread blocks on two SMs work on one tcgen05 MMA (cta_group::2).
//
// Work unit: (item, kv head, two consecutive M-tiles), one M-tile per CTA of the pair.  An M-tile is 128 query rows
// = floor(128 / g) consecutive chunk tokens x the g query heads that share the kv head.  The pair walks the keys its
// rows can see (the cached prefix, then the chunk itself up to the diagonal) in tiles of 128 keys.  Per key tile j:
//
//   S = Q K^T      one MMA of M 256 x N 128 x K 128 for the pair.  Each CTA supplies its own 128 rows of Q and HALF of
//                  the tile's keys (64) from its own shared memory and receives its 128 x 128 scores in its own tensor
//                  memory: per MMA step an SM reads 4 KB of Q and 2 KB of K for 64 cycles of math, where one CTA
//                  alone with 64-key tiles read 6 KB per 32 cycles and was held by its shared-memory port.  Two S
//                  buffers, so S(j+1) is computed while the softmax of tile j runs.
//   softmax        two warpgroups per CTA, each with its own KEY STREAM: warpgroup w takes keys 64 w .. 64 w + 63 of
//                  every tile, one thread per query row: tcgen05.ld its 64 scores, P = exp2(scale * s - m) as packed
//                  bf16 stored back over the start of its half of the S buffer, row sum.  A stream has its own
//                  reference max, row sum and O accumulator, so the two warps that share a row (they sit on the same
//                  SM sub-partition: tensor-memory lanes are tied to warp % 4) never exchange anything while the keys
//                  stream by; the two streams are merged once, at the end.  After a stream's first tile m is not
//                  recomputed per tile: the exponentials are taken against the current reference max, and only a row
//                  sum that explodes (or a masked tile) sends the tile down the careful path (row max, new reference,
//                  the stream's O rescaled in tensor memory).  One pair of exponentials in kPolyOneIn is evaluated
//                  on the FMA pipe.
//   O_w += P_w V   per stream an MMA of M 256 x N 128 x K 64 with the A operand (P) in tensor memory; each CTA supplies
//                  HALF of V's dims (64) for the keys, straight from the [key][dim] page layout (MN-major B).
//
// Roles per CTA (12 warps): warp 0 copies Q and the CTA's half of every K tile, warp 3 its half of every V tile (TMA,
// one box per page; page ids fetched 32 at a time, a batch ahead); warp 2 waits for each landed tile, zeroes the V
// rows of dead keys in the last tile and tells the leader that this CTA's half is ready; warp 1 of the leader (the
// even CTA) issues every MMA (the whole warp walks the loop so that descriptors are warp-uniform values; one elected
// lane issues); warps 4-7 and 8-11 are the softmax warpgroups, which also write the result.
// Completion of MMAs reaches both CTAs through tcgen05.commit to the barriers of both; all other cross-CTA signals are
// mbarrier arrivals at the leader.  No load is multicast: each CTA copies what it needs itself.
// A CTA uses ~194 KB of shared memory (Q 32 KB, 10 K/V stages of 16 KB) and all 512 tensor-memory columns (two S
// buffers of 128, two O accumulators of 128).
// Every wait is a bounded mbarrier poll; a pair in which any wait ran out tells both CTAs and runs to its end.
#include <cuda.h>

#include <climits>
#include <type_traits>

#include "rollart_internal.cuh"
#include "tc_ptx.cuh"

namespace rollart {

namespace {

using namespace tc;

constexpr int kRows = 128;                 // query rows of a CTA (the pair's MMA has M = 256)
constexpr int kKeys = 128;                 // keys per KV tile
constexpr int kOwnKeys = kKeys / 2;        // keys of a K tile held by one CTA
constexpr int kOwnDims = kHeadDim / 2;     // dims of a V tile held by one CTA
constexpr int kStages = 10;                // ring of stages; K(j) and V(j) take alternate slots
constexpr int kThreads = 384;
constexpr int kCols = kKeys / 2;           // S columns (keys) of a tile per softmax thread: one key stream per warpgroup
constexpr int kMaxItems = kChunkItemsPerLaunch;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.f;   // log2 units
constexpr float kRowSumLimit = 16777216.f; // 2^24: a half-row sum above this sends the tile down the careful path
constexpr int kPolyOneIn = 3;              // one pair of exponentials in this many goes to the FMA pipe

constexpr int kHalfQ = kRows * 128;        // 16 KB: 128 rows x 64 dims
constexpr int kTileQ = 2 * kHalfQ;         // [dim half][row][128 B]
constexpr int kHalfK = kOwnKeys * 128;     // 8 KB: 64 keys x 64 dims
constexpr int kStageBytes = 2 * kHalfK;    // K: [dim half][key][128 B]; V: [key (128)][128 B = the CTA's 64 dims]
static_assert(kStageBytes == kKeys * kOwnDims * 2, "a V half tile fills a stage exactly");
constexpr int kOffQ = 0;
constexpr int kOffKV = kOffQ + kTileQ;
constexpr int kOffBars = kOffKV + kStages * kStageBytes;
constexpr int kNumBars = 2 + 3 * kStages + 10;  // q_full, q_ready | full, empty, ready per stage | s_full per S buffer | p_full, o_done per key stream and S buffer
constexpr int kOffTmemSlot = kOffBars + kNumBars * 8;
constexpr int kOffAbort = kOffTmemSlot + 8;
constexpr int kOffFatal = kOffAbort + 8;                   // the leader's reading of the status word's fatal flag
constexpr int kOffXMl = kOffFatal + 8;                     // [stream][row]: (m, l) of each key stream, for the final merge
constexpr int kSmemUsed = kOffXMl + 2 * kRows * 8;
constexpr int kSmemBytes = kSmemUsed + 1024;               // + slack for the 1024-byte alignment
static_assert(kSmemBytes <= 227 * 1024, "one block must fit an SM");
static_assert((kMaxItems + 1) * 4 + kMaxItems * 16 <= kStages * kStageBytes, "the tile prefix and the item table are staged in the KV stages");
static_assert(kStages % 2 == 0, "K tiles and V tiles alternate in the ring");

constexpr int kTmemCols = 512;             // S buffer b at columns b * 128; stream w's P over the first 32 columns of its half (64 w ..) of the S buffer
constexpr int kTmemO = 256;                // O of stream w at 256 + 128 w

struct PairParams {
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
    DeviceStatus *status;
};

// Bounded wait on a barrier of this CTA (its arrivals may come from the other CTA).  A wait that runs out raises the
// abort flag of both CTAs; from then on nobody in the pair waits, every role runs its bounded loops to the end.
__device__ __forceinline__ void pair_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t peer_abort,
                                          DeviceStatus *status, int where) {
    constexpr long long kWaitCycles = 2000000000LL;   // about a second
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
        st_cluster_u32(peer_abort, 1u);
        report(status, ROLLART_ERR_TIMEOUT, where, 3);
        status->fatal = 1;         // later pairs of this launch do not start
    }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
chunk_attn_pair_kernel(const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap kmap,
                       const __grid_constant__ CUtensorMap vmap, const PairParams prm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hkv = prm.num_kv_heads, P = prm.page_size, g = prm.group;
    const int tpt = kRows / g;                       // chunk tokens per M-tile
    const uint32_t rank = cluster_ctarank();         // 0: the leader, which issues the MMAs
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + kOffAbort);
    volatile int *s_fatal = reinterpret_cast<volatile int *>(smem + kOffFatal);
    volatile uint32_t *s_tmem = reinterpret_cast<volatile uint32_t *>(smem + kOffTmemSlot);
    int *s_prefix = reinterpret_cast<int *>(smem + kOffKV);    // staged in the KV stages during the prologue

    if (static_cast<int>(smem - smem_raw) + kSmemUsed > kSmemBytes) {   // cannot happen: the slack covers any alignment
        if (threadIdx.x == 0) report(prm.status, ROLLART_ERR_CUDA, static_cast<int>(smem - smem_raw), 3);
        return;
    }
    const uint32_t bars = smem_u32(smem + kOffBars);
    const uint32_t bar_qfull = bars, bar_qready = bars + 8u;
    // ring slot r (K(j) is r = 2j, V(j) is r = 2j + 1) lives in stage r % kStages
    auto bar_full = [&](int s) { return bars + 8u * (2 + s); };                  // this CTA's copies have landed
    auto bar_empty = [&](int s) { return bars + 8u * (2 + kStages + s); };       // the MMAs that read the stage are done
    auto bar_ready = [&](int s) { return bars + 8u * (2 + 2 * kStages + s); };   // leader: both CTAs' halves are in place
    auto bar_sfull = [&](int b) { return bars + 8u * (2 + 3 * kStages + b); };
    auto bar_pfull = [&](int w, int b) { return bars + 8u * (2 + 3 * kStages + 2 + 2 * w + b); };   // leader: stream w's P of both CTAs is stored
    auto bar_odone = [&](int w, int b) { return bars + 8u * (2 + 3 * kStages + 6 + 2 * w + b); };
    const uint32_t peer_abort = map_to_cta(smem_u32(smem + kOffAbort), rank ^ 1u);

    // ---- set-up that does not depend on the unit, first: it overlaps the loads of the item table below ----
    // barriers (one per thread), Q zero fill (rows beyond tpt * g are never written by the copy), tensor memory
    if (threadIdx.x < kNumBars) {
        const int i = static_cast<int>(threadIdx.x);
        uint32_t count = 1;                                                      // q_full, full, empty, s_full, o_done
        if (i == 1 || (i >= 2 + 2 * kStages && i < 2 + 3 * kStages)) count = 2;  // q_ready, ready: one arrival per CTA
        else if (i >= 2 + 3 * kStages + 2 && i < 2 + 3 * kStages + 6) count = 8; // p_full: 4 warps x 2 CTAs
        mbar_init(bars + 8u * i, count);
    }
    if (threadIdx.x == 0) {
        *s_abort = 0;
        // an earlier block ran out of patience: the leader's reading of the flag decides for the pair
        s_fatal[0] = *reinterpret_cast<volatile int *>(&prm.status->fatal) != 0 ? 1 : 0;
    }
    for (int i = threadIdx.x; i < kTileQ / 16; i += kThreads) reinterpret_cast<uint4 *>(smem + kOffQ)[i] = make_uint4(0, 0, 0, 0);
    if (warp == 0) tmem_alloc_pair(smem_u32(smem + kOffTmemSlot), kTmemCols);

    // ---- which (item, kv head, pair of M-tiles) is this cluster?  pairs per item -> prefix -> search.  The same pass
    //      keeps every item's rows, trajectory and length in shared memory, so that the unit's geometry below needs no
    //      further (dependent) global loads ----
    int *s_item = s_prefix + (kMaxItems + 1);             // [item][4]: first row, rows, trajectory, length (-1: invalid trajectory)
    for (int i = threadIdx.x; i < prm.n_items; i += kThreads) {
        const int q0 = __ldg(prm.q_indptr + i), n = __ldg(prm.q_indptr + i + 1) - q0;
        const int t = prm.traj_ids ? __ldg(prm.traj_ids + i) : i + prm.item_offset;
        s_item[4 * i] = q0; s_item[4 * i + 1] = n; s_item[4 * i + 2] = t;
        s_item[4 * i + 3] = (t >= 0 && t < prm.num_traj) ? __ldg(prm.seq_lens + t) : -1;
        s_prefix[i + 1] = n > 0 ? (n + 2 * tpt - 1) / (2 * tpt) : 0;
    }
    if (threadIdx.x == 0) s_prefix[0] = 0;
    __syncthreads();
    if (warp == 1) {        // inclusive scan of the pair counts, in place (warp 0 is allocating tensor memory)
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
    const int unit = static_cast<int>(blockIdx.x >> 1);      // both CTAs of a cluster
    const int total_units = s_prefix[prm.n_items] * hkv;
    int item = 0, head = 0, pair = 0;
    if (unit < total_units) {
        int lo = 0, hi = prm.n_items;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_prefix[mid] * hkv <= unit) lo = mid; else hi = mid;
        }
        item = lo;
        const int np = max(1, s_prefix[lo + 1] - s_prefix[lo]);
        const int rem = unit - s_prefix[lo] * hkv;
        head = rem / np;
        pair = np - 1 - (rem - head * np);      // later M-tiles see more keys: start the longest ones first
    }

    // ---- geometry of this unit.  Whether the pair has work depends on the unit alone, so both CTAs decide alike ----
    bool active = unit < total_units;
    const int q_row0 = s_item[4 * item], n_chunk = s_item[4 * item + 1], t = s_item[4 * item + 2];
    int L = s_item[4 * item + 3];
    if (active) {
        int bad_value = 0;
        bool bad = false;
        if (q_row0 < 0 || n_chunk < 0 || static_cast<long long>(q_row0) + n_chunk > prm.total_q) { bad = true; bad_value = q_row0; }   // q_indptr does not describe rows of q
        else if (t < 0 || t >= prm.num_traj) { bad = true; bad_value = t; }
        else if (L < 0 || L > prm.max_seq_len || n_chunk > L) { bad = true; bad_value = L; }
        if (bad) {
            if (threadIdx.x == 0 && rank == 0) report(prm.status, ROLLART_ERR_BOUNDS, bad_value, 3);
            active = false;
        }
    }
    if (!active) L = 0;
    const int prior = L - n_chunk;
    const int first_tok = (2 * pair + static_cast<int>(rank)) * tpt;       // first chunk token of this CTA's M-tile
    const int toks = max(0, min(tpt, n_chunk - first_tok));                // its live tokens (the second CTA may have none)
    const int pair_toks_end = min(n_chunk, (2 * pair + 2) * tpt);          // one past the pair's last live token
    const int nmax = (prior + pair_toks_end + kKeys - 1) / kKeys;          // key tiles of the pair (>= 1)
    const int min_count = min(L, prior + first_tok + 1);                   // keys the CTA's first row sees
    const int32_t *table_row = prm.page_table + static_cast<long long>(active ? t : 0) * prm.max_pages;

    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();             // the zeroed Q rows are ordered before the copy that lands beside them
    tc_fence_before();
    __syncthreads();                 // everyone has read the tables: the KV stages are free again
    cluster_sync_all();              // both CTAs' barriers exist before anything arrives on them
    tc_fence_after();
    const uint32_t tmem = *s_tmem;
    // (the leader stays resident until the pair's last common barrier, so its shared memory may be read here)
    const bool run = active && ld_cluster_u32(map_to_cta(smem_u32(smem + kOffFatal), 0)) == 0u;

    if (!run) {
        // fall through to the common exit
    } else if (warp == 0 || warp == 3) {
        // =============================== copy warps ===============================
        // Warp 0 brings Q and this CTA's 64 keys of every K tile (two boxes per page: 64 dims each); warp 3 brings its
        // 64 dims of every V tile (one box per page).  Both use the [rows][128 dims] view of a pool.
        const int kv = warp == 3 ? 1 : 0;
        if (kv == 0 && lane == 0) {
            if (toks > 0) {
                mbar_arrive_expect_tx(bar_qfull, static_cast<uint32_t>(tpt * g) * kRowBytes);
                const uint32_t dst = smem_u32(smem + kOffQ);
                tma_load_3d(dst, &qmap, bar_qfull, 0, head * g, q_row0 + first_tok);
                tma_load_3d(dst + kHalfQ, &qmap, bar_qfull, 64, head * g, q_row0 + first_tok);
            } else {
                mbar_arrive(bar_qfull);      // no live row here: Q stays zero
            }
        }
        const int pages_per_tile = kKeys / P;
        const int my_pages = kv == 0 ? kOwnKeys / P : pages_per_tile;            // boxes this warp issues per tile
        const int my_first = kv == 0 ? static_cast<int>(rank) * (kOwnKeys / P) : 0;
        const int tiles_per_batch = 32 / pages_per_tile;
        const uint32_t box_bytes = static_cast<uint32_t>(P) * 128;                // P rows x 64 dims
        // Page ids are fetched 32 at a time, one per lane, and the next 32 are requested a whole batch ahead, so the
        // table lookup (a dependent load) is off the copy loop's path.
        auto load_ids = [&](int batch) {
            const int lp = batch * 32 + lane;
            int pg = -1;
            if (lp * P < L && lp < prm.max_pages) {
                pg = __ldg(table_row + lp);
                if (pg < 0 || pg >= prm.num_pages) {
                    if (kv == 1 && rank == 0) report(prm.status, ROLLART_ERR_BOUNDS, pg, 3);
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
            int pg = __shfl_sync(0xffffffffu, ids_cur, (within * pages_per_tile + my_first + lane) & 31);
            if (lane >= my_pages) pg = -1;
            const uint32_t nvalid = __popc(__ballot_sync(0xffffffffu, pg >= 0));
            const int r = 2 * j + kv, stage = r % kStages;
            pair_wait(bar_empty(stage), ((r / kStages) & 1) ^ 1, s_abort, peer_abort, prm.status, 1 + kv);
            if (lane == 0) mbar_arrive_expect_tx(bar_full(stage), nvalid * (kv == 0 ? 2u : 1u) * box_bytes);
            __syncwarp();
            if (pg >= 0) {
                const uint32_t dst = smem_u32(smem + kOffKV + stage * kStageBytes) + lane * box_bytes;
                const int row = (pg * hkv + head) * P;
                if (kv == 0) {
                    tma_load_2d(dst, &kmap, bar_full(stage), 0, row);
                    tma_load_2d(dst + kHalfK, &kmap, bar_full(stage), 64, row);
                } else {
                    tma_load_2d(dst, &vmap, bar_full(stage), kOwnDims * static_cast<int>(rank), row);
                }
            }
        }
    } else if (warp == 2) {
        // =============================== stage warp ===============================
        // Waits for this CTA's copies of each ring slot and tells the leader.  In the last V tile the rows of keys at or
        // beyond L (dead slots of the last page, pages that were never copied) are zeroed first: their P is exactly 0,
        // but 0 x NaN would still poison O.
        const uint32_t leader_qready = map_to_cta(bar_qready, 0);
        pair_wait(bar_qfull, 0, s_abort, peer_abort, prm.status, 5);
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(leader_qready);
        for (int r = 0; r < 2 * nmax; ++r) {
            const int stage = r % kStages;
            pair_wait(bar_full(stage), (r / kStages) & 1, s_abort, peer_abort, prm.status, 6 + (r & 1));
            const int key0 = (r >> 1) * kKeys;
            if ((r & 1) && key0 + kKeys > L) {
                const uint32_t v_addr = smem_u32(smem + kOffKV + stage * kStageBytes);
                const int first_dead = max(0, L - key0);
                for (int idx = lane; idx < (kKeys - first_dead) * 8; idx += 32) {
                    const uint32_t a = v_addr + static_cast<uint32_t>(first_dead + (idx >> 3)) * 128u + static_cast<uint32_t>(idx & 7) * 16u;
                    asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0) : "memory");
                }
                fence_proxy_async();      // the zeroed rows become visible to the tensor core's reads
            }
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(bar_ready(stage), 0));
        }
    } else if (warp == 1) {
        // =============================== MMA warp (leader only) ===============================
        // One thread issues QK(0) | QK(j+1) PV(j) | ...: S of the next key tile is ready before the softmax of this one
        // ends.  MMAs run in issue order, which is what protects the reuse of an S buffer (it holds P(j-1) until
        // PV(j-1), issued before QK(j+1), has read it).
        // The whole warp walks the loop (waits, descriptor arithmetic: warp-uniform values, which the compiler can keep
        // in uniform registers, where the MMA instruction takes its operands from); only the MMA and commit
        // instructions themselves are predicated on one elected lane.
        if (rank == 0) {
            constexpr uint32_t kIdescQK = idesc(2 * kRows, kKeys, false);
            constexpr uint32_t kIdescPV = idesc(2 * kRows, kHeadDim, true);
            const bool elected = elect_one();
            const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
            const uint32_t kv_addr = smem_u32(smem + kOffKV);
            const uint64_t q_desc = smem_desc(smem_u32(smem + kOffQ), 16);
            auto ready_wait = [&](int r, int where) {
                pair_wait(bar_ready(r % kStages), (r / kStages) & 1, s_abort, peer_abort, prm.status, where);
            };
            auto issue_qk = [&](int j) {
                ready_wait(2 * j, 8);                       // K(j), both halves
                tc_fence_after();
                const uint64_t k_desc = smem_desc(kv_addr + ((2 * j) % kStages) * kStageBytes, 16);
                const uint32_t s_tm = tm + (j & 1) * kKeys;
#pragma unroll
                for (int ks = 0; ks < kHeadDim / 16; ++ks) {   // 16 dims per step; the second 64 dims live in the other half
                    const uint64_t qoff = static_cast<uint64_t>(((ks >> 2) * kHalfQ + (ks & 3) * 32) >> 4);
                    const uint64_t koff = static_cast<uint64_t>(((ks >> 2) * kHalfK + (ks & 3) * 32) >> 4);
                    if (elected) umma_pair_bf16(s_tm, q_desc + qoff, k_desc + koff, kIdescQK, ks > 0 ? 1u : 0u);
                }
                if (elected) {
                    umma_pair_commit(bar_sfull(j & 1));
                    umma_pair_commit(bar_empty((2 * j) % kStages));
                }
                __syncwarp();
            };
            pair_wait(bar_qready, 0, s_abort, peer_abort, prm.status, 9);
            issue_qk(0);
            for (int j = 0; j < nmax; ++j) {
                if (j + 1 < nmax) issue_qk(j + 1);
                ready_wait(2 * j + 1, 10);                  // V(j), both halves
                // V half tile is [key][128 B]: the 16 keys of step ks start 2 KB further on; 8-key groups are 1 KB apart
                const uint64_t v_desc = smem_desc(kv_addr + ((2 * j + 1) % kStages) * kStageBytes, 1024);
                const uint32_t p_tm = tm + (j & 1) * kKeys;
                const uint32_t acc0 = j > 0 ? 1u : 0u;
#pragma unroll
                for (int w = 0; w < 2; ++w) {               // the two key streams: keys 64 w .. 64 w + 63 of the tile into O_w
                    pair_wait(bar_pfull(w, j & 1), (j >> 1) & 1, s_abort, peer_abort, prm.status, 11);
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < kCols / 16; ++ks)     // 16 keys per step: 8 packed columns of P's row
                        if (elected)
                            umma_pair_bf16_ts(tm + kTmemO + w * kHeadDim, p_tm + w * kCols + ks * 8,
                                              v_desc + static_cast<uint64_t>(((w * kCols + ks * 16) * 128) >> 4), kIdescPV,
                                              ks > 0 ? 1u : acc0);
                    if (elected) {
                        if (w == 1) umma_pair_commit(bar_empty((2 * j + 1) % kStages));
                        umma_pair_commit(bar_odone(w, j & 1));
                    }
                    __syncwarp();
                }
            }
        }
        __syncwarp();
    } else {
        // =============================== softmax warpgroups ===============================
        // Warpgroup w owns key stream w: keys 64 w .. 64 w + 63 of every tile, with its own reference max, row sum and
        // O accumulator, so the two warps that share a row never have to agree on anything while the keys stream by;
        // the two streams are merged once, at the end.
        const int wg = (warp - 4) >> 2;
        const int quarter = warp & 3;                         // tensor-memory lanes 32 * quarter .. + 31 belong to this warp
        const int row = quarter * 32 + lane;
        const uint32_t lane_addr = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        const uint32_t s_addr = lane_addr + wg * kCols, o_addr = lane_addr + kTmemO + wg * kHeadDim;
        const int tok_local = row / g, head_local = row - tok_local * g;
        const bool live = tok_local < toks;
        const int count = min(L, prior + first_tok + min(tok_local, max(toks, 1) - 1) + 1);   // keys this row sees (>= 1)
        const float scale = prm.scale_log2;
        const uint32_t leader_pfull = map_to_cta(bar_pfull(wg, 0), 0);
        float m_ref = -INFINITY, l_sum = 0.f;

        for (int j = 0; j < nmax; ++j) {
            const int sb = j & 1;
            const uint32_t sbuf = s_addr + sb * kKeys;
            pair_wait(bar_sfull(sb), (j >> 1) & 1, s_abort, peer_abort, prm.status, 12);
            tc_fence_after();
            uint32_t sraw[2][32];
            tmem_ld32(sbuf, sraw[0]);
            tmem_ld32(sbuf + 32, sraw[1]);
            tmem_wait_ld();

            const int key0 = j * kKeys;
            const bool need_mask = key0 + kKeys > min_count;    // the same for every thread of the CTA
            const int live_keys = count - key0 - wg * kCols;    // of this thread's 64 columns, those the row sees
            float rs[4];
            // two copies of the pass, chosen once per tile: the unmasked one carries no compare / select per element
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
                        if (kPoly && ((h * 16 + (c >> 1)) % kPolyOneIn) == kPolyOneIn - 1) {
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
                    // P as the next A operand: 32 keys of this row as 16 packed columns at the start of this stream's half of the S buffer
                    tmem_st16(sbuf + h * 16, packed);
                }
                return (rs[0] + rs[1]) + (rs[2] + rs[3]);
            };
            // Fast path (every unmasked tile after the first): no max pass.  The exponentials are taken against the
            // stream's reference max m_ref (the max of some earlier score, so later keys far below it rightly vanish);
            // keys far above it make the row sum explode, and then (rarely) the tile is redone the careful way below.
            // Up to that bound P and the sums just carry a larger exponent: fp32 accumulation and the 8-bit mantissa
            // of bf16 P lose nothing by it.
            float rsum = 0.f, corr = 1.f;
            bool careful = j == 0 || need_mask;
            if (!careful) {
                rsum = exp_pass(std::false_type{}, std::true_type{}, -m_ref);
                // also true for inf / NaN, and for a score so far above the reference that the FMA-pipe exponential broke
                careful = __any_sync(0xffffffffu, !(rsum <= kRowSumLimit) || poly_top > kPolyArgTop);
                if (careful) tmem_wait_st();      // the stores of the abandoned pass land before the new ones
            }
            if (careful) {
                float rmax;
                if (!need_mask) {
                    // the max of scale * s is scale * (max or min of s): the extreme of the raw scores, 8 chains of 3-input ops
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
                    // masked tile: keys the row does not see are left out (their scores may be anything); a row that sees
                    // none of this stream's keys keeps rmax = -inf and stores P = 0
                    rmax = -INFINITY;
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (h * 32 + c < live_keys) rmax = fmaxf(rmax, __uint_as_float(sraw[h][c]) * scale);
                }
                // the reference max moves only when it has to (first keys of the stream) or when a row outgrew it by 2^8
                const bool grow = rmax > m_ref + kRescaleThreshold;
                const float m_new = grow ? rmax : m_ref;
                corr = grow ? ex2(m_ref - m_new) : 1.f;   // ex2(-inf) = 0 while the stream has seen nothing
                if (j >= 1 && __any_sync(0xffffffffu, grow)) {
                    // rare: some row of this warp moved its reference max, so this stream's O (the tiles before this
                    // one) must be rescaled before PV of this tile; PV of the previous tile has to be finished first
                    pair_wait(bar_odone(wg, (j - 1) & 1), ((j - 1) >> 1) & 1, s_abort, peer_abort, prm.status, 13);
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
                // a stream that has not seen a key yet (m_ref = -inf) stores zeros through the masked pass
                // (every exponential on the special-function unit here: the careful path has no bound on its arguments to rely on)
                rsum = need_mask ? exp_pass(std::true_type{}, std::false_type{}, -m_ref)
                                 : exp_pass(std::false_type{}, std::false_type{}, -m_ref);
            }
            l_sum = l_sum * corr + rsum;
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_pfull + 8u * sb);
        }

        // ---- epilogue: merge the two streams, O / l -> bf16 rows of out; warpgroup w writes dims 64 w .. 64 w + 63 ----
        pair_wait(bar_odone(0, (nmax - 1) & 1), ((nmax - 1) >> 1) & 1, s_abort, peer_abort, prm.status, 14);
        pair_wait(bar_odone(1, (nmax - 1) & 1), ((nmax - 1) >> 1) & 1, s_abort, peer_abort, prm.status, 14);
        tc_fence_after();
        volatile float *x_ml = reinterpret_cast<volatile float *>(smem + kOffXMl);
        x_ml[(wg * kRows + row) * 2] = m_ref;
        x_ml[(wg * kRows + row) * 2 + 1] = l_sum;
        named_bar_sync(1 + quarter, 64);                      // the two warps that share these rows
        const float m0 = x_ml[row * 2], l0 = x_ml[row * 2 + 1], m1 = x_ml[(kRows + row) * 2], l1 = x_ml[(kRows + row) * 2 + 1];
        const float m_all = fmaxf(m0, m1);
        const float w0 = m0 == -INFINITY ? 0.f : ex2(m0 - m_all), w1 = m1 == -INFINITY ? 0.f : ex2(m1 - m_all);
        const float l_all = l0 * w0 + l1 * w1;
        const float inv = l_all > 0.f ? prm.out_scale / l_all : 0.f;
        const float f0 = w0 * inv, f1 = w1 * inv;
        const uint32_t o_both = lane_addr + kTmemO + wg * kCols;      // this warpgroup's 64 dims, in O_0; O_1 is 128 columns on
        const long long orow = (static_cast<long long>(q_row0 + first_tok + tok_local) * prm.num_q_heads + head * g + head_local);
#pragma unroll 1
        for (int c0 = 0; c0 < kCols; c0 += 32) {
            uint32_t oa[32], ob[32];
            tmem_ld32(o_both + c0, oa);
            tmem_ld32(o_both + kHeadDim + c0, ob);
            tmem_wait_ld();
            if (live) {
                float ov[32];
#pragma unroll
                for (int k = 0; k < 32; ++k) ov[k] = fmaf(__uint_as_float(ob[k]), f1, __uint_as_float(oa[k]) * f0);
                uint4 *dst = reinterpret_cast<uint4 *>(prm.out + orow * kHeadDim + wg * kCols + c0);
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
        if (live && wg == 0 && prm.lse != nullptr) prm.lse[orow] = l_all > 0.f ? (m_all + log2f(l_all)) * kLn2 : -INFINITY;
    }

    // ---- all roles of both CTAs meet (nothing of the pair is in flight any more); the tensor memory goes back ----
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc_pair(tmem, kTmemCols);
    }
}

}  // namespace

cudaError_t launch_chunk_attn_pair(const AttnCall &c, cudaStream_t stream, int64_t *launches) {
    const int hkv = c.pool.num_kv_heads, g = c.num_q_heads / hkv, tpt = kRows / g;
    cudaError_t e = cudaFuncSetAttribute(chunk_attn_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    CUtensorMap qmap, kmap, vmap;
    if (!encode_q_map(&qmap, c.q, c.total_q, c.num_q_heads, g) ||
        !encode_pool_rows(&kmap, c.pool.k, c.pool.num_pages, hkv, c.pool.page_size) ||
        !encode_pool_rows(&vmap, c.pool.v, c.pool.num_pages, hkv, c.pool.page_size))
        return cudaErrorInvalidValue;
    for (int base = 0; base < c.n_items; base += kMaxItems) {
        const int n = c.n_items - base < kMaxItems ? c.n_items - base : kMaxItems;
        PairParams prm;
        prm.page_table = c.trajs.page_table; prm.seq_lens = c.trajs.seq_lens;
        prm.traj_ids = c.traj_ids ? c.traj_ids + base : nullptr;
        prm.q_indptr = c.q_indptr + base;
        prm.max_pages = c.trajs.max_pages; prm.num_traj = c.trajs.num_traj; prm.num_pages = c.pool.num_pages;
        prm.page_size = c.pool.page_size; prm.num_kv_heads = hkv; prm.num_q_heads = c.num_q_heads; prm.group = g;
        prm.n_items = n; prm.item_offset = base; prm.max_seq_len = c.max_seq_len; prm.total_q = c.total_q;
        prm.out = c.out; prm.lse = c.lse; prm.scale_log2 = c.sm_scale * kLog2e; prm.out_scale = c.v_scale; prm.status = c.status;
        // an upper bound on the M-tile pairs of these items: every item has at most one ragged pair
        const long long pairs = (static_cast<long long>(c.total_q) + 2 * tpt - 1) / (2 * tpt) + n;
        const long long blocks = 2 * pairs * hkv;
        if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
        chunk_attn_pair_kernel<<<static_cast<unsigned>(blocks), kThreads, kSmemBytes, stream>>>(qmap, kmap, vmap, prm);
        ++*launches;
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace rollart
