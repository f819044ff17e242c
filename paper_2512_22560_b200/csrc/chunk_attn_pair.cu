// Observation-chunk attention on CTA pairs: two thread blocks on two SMs work on one tcgen05 MMA (cta_group::2).
//
// Work unit: (item, kv head, two consecutive M-tiles), one M-tile per CTA of the pair.  An M-tile is 128 query rows
// = floor(128 / g) consecutive chunk tokens x the g query heads that share the kv head.  The pair walks the keys its
// rows can see (the cached prefix, then the chunk itself up to the diagonal) in tiles of 128 keys.  Per key tile j:
//
//   S = Q K^T      one MMA of M 256 x N 128 x K 128 for the pair.  Each CTA supplies its own 128 rows of Q and HALF of
//                  the tile's keys (64) from its own shared memory and receives its 128 x 128 scores in its own tensor
//                  memory: per MMA step an SM reads 4 KB of Q and 2 KB of K for 64 cycles of math, where one CTA
//                  alone with 64-key tiles read 6 KB per 32 cycles and was held by its shared-memory port.  THREE S
//                  buffers: S(j+3) is issued right behind PV(j), so the chain "P(j) stored -> PV(j) -> S of the tile
//                  that reuses the buffer -> its softmax" spans three tiles and its signalling latencies stay off the
//                  critical path (with two buffers they were a quarter of a tile's time).
//   softmax        two warpgroups per CTA that take the key tiles in turn (warpgroup w the tiles j = w mod 2), one
//                  thread per query row with all 128 scores of the row: tcgen05.ld in four quarters of 32 columns,
//                  each load in flight behind the arithmetic of the quarter before; P = exp2(scale * s - m) as packed
//                  bf16 stored back over the start of the S buffer; row sum.  The two warps of an SM sub-partition work
//                  on different tiles, so each one's waits fall into the other's arithmetic, and the fixed cost of a
//                  tile (barrier, fences, hand-over) is paid once per 128 columns.
//                  The reference m of a row is fixed after the first tile (the max of the row's visible scores there;
//                  every row sees key 0) and never moves: P and the sums of a row whose later scores are larger just
//                  carry a larger exponent, which fp32 accumulation and bf16's 8-bit mantissa do not mind.  So there
//                  is no rescaling of O, one O accumulator serves both warpgroups, and the freed tensor-memory columns
//                  hold the third S buffer.  A row sum of a tile beyond 2^64 (scores more than ~44 nats above the
//                  first tile's max, or inf / NaN), or an argument beyond the range of the FMA-pipe exponential,
//                  marks the unit in a bitmap; marked units are computed again by the single-CTA kernel, which moves
//                  its reference max, in a launch that follows this one (its other blocks return at once).
//                  One pair of exponentials in kPolyOneIn is evaluated on the FMA pipe.
//   O += P V       an MMA of M 256 x N 128 x K 128 with the A operand (P) in tensor memory; each CTA supplies HALF of
//                  V's dims (64) for the keys, straight from the [key][dim] page layout (MN-major B).
//
// The pairs are persistent: one cluster per two SMs walks units handed out in order from a counter in global memory
// (warp 1 of the second CTA, which issues no MMAs, draws the numbers and puts them into a small ring in both CTAs'
// shared memory).  Barrier phases, the K/V ring and the S buffers run on from unit to unit, so the copies of the next
// unit and its first three QK run while the softmax warps write the last one out; the barriers, the tensor-memory
// allocation and the item tables are set up once per CTA.  Two more barriers order the reuse of what a unit owns alone:
// Q (free once the unit's last QK is done) and O (free once every softmax warp of the pair has read it).
//
// Roles per CTA (16 warps).  Copies: a TMA copy costs the warp that issues it ~135 cycles whatever its size, and a
// tile of 16-slot pages needs 12 of them per CTA (4 K pages with both 64-dim halves in one 4-D box, 8 V pages), so they
// are spread: warps 0 and 15 copy the CTA's half of every K tile (warp 0 also Q), warps 3, 12, 13, 14 its half of
// every V tile, each at least two pages of a tile (with larger pages fewer of them take part); page ids are fetched 32
// at a time, a batch ahead.  Warp 2 waits for each landed tile, zeroes the V rows of dead keys in the last tile and
// tells the leader that this CTA's half is ready; warp 1 of the leader (the even CTA) issues every MMA (the whole
// warp walks the loop so that descriptors are warp-uniform values; one elected lane issues); warps 4-7 and 8-11 are
// the softmax warpgroups, which also write the result.
// Completion of MMAs reaches both CTAs through tcgen05.commit to the barriers of both; all other cross-CTA signals are
// mbarrier arrivals at the leader.  No load is multicast: each CTA copies what it needs itself.
// A CTA uses ~215 KB of shared memory (Q 32 KB, 6 K stages and 4 V stages of 16 KB, 20 KB of item tables) and all 512 tensor-memory columns
// (three S buffers of 128, one O accumulator of 128).
// Every wait is a bounded mbarrier poll; a pair in which any wait ran out tells both CTAs and runs to its end.
#include <cuda.h>

#include <algorithm>
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
constexpr int kStagesK = 6;                // ring of K stages: K(j) in stage j % 6 (QK runs three tiles ahead of PV)
constexpr int kStagesV = 4;                // ring of V stages: V(j) in stage 6 + j % 4
constexpr int kStages = kStagesK + kStagesV;
constexpr int kSBufs = 3;                  // S buffers in tensor memory
constexpr int kSoftmaxGroups = 2;          // softmax warpgroups: group w takes the key tiles j = w (mod 2), whole
constexpr int kVCopyWarps = 4;             // warps that may share the V copies of a tile (warp 3 and warps 12..14)
constexpr int kKCopyWarps = 2;             // likewise for the K copies (warp 0 and warp 15)
constexpr int kThreads = 128 + 128 * kSoftmaxGroups + 32 * (kVCopyWarps - 1) + 32 * (kKCopyWarps - 1);
constexpr int kMaxItems = kChunkItemsPerLaunch;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRowSumLimit = 18446744073709551616.f;   // 2^64: a row sum of one tile above this marks the unit for the careful kernel
constexpr int kPolyOneIn = 8;              // one pair of exponentials in this many goes to the FMA pipe

constexpr int kHalfQ = kRows * 128;        // 16 KB: 128 rows x 64 dims
constexpr int kTileQ = 2 * kHalfQ;         // [dim half][row][128 B]
constexpr int kHalfK = kOwnKeys * 128;     // 8 KB: 64 keys x 64 dims
constexpr int kStageBytes = 2 * kHalfK;    // K: [group of 8 keys][dim half][key in group][128 B]; V: [key (128)][128 B = the CTA's 64 dims]
static_assert(kStageBytes == kKeys * kOwnDims * 2, "a V half tile fills a stage exactly");
constexpr int kOffQ = 0;
constexpr int kOffKV = kOffQ + kTileQ;
constexpr int kOffBars = kOffKV + kStages * kStageBytes;
constexpr int kUnitRing = 4;               // units handed out ahead of the slowest role
constexpr int kNumBars = 2 + 3 * kStages + 2 * kSBufs + 3 + 2 * kUnitRing;  // q_full, q_ready | full, empty, ready per stage | s_full, p_full per S buffer | o_done, q_free, o_free | unit_full, unit_empty per ring slot
constexpr int kOffTmemSlot = kOffBars + kNumBars * 8;
constexpr int kOffAbort = kOffTmemSlot + 8;
constexpr int kOffFatal = kOffAbort + 8;                   // the leader's reading of the status word's fatal flag
constexpr int kOffXMl = kOffFatal + 8;                     // [row]: the row's reference max; then [warpgroup][row]: the row sums
constexpr int kOffTable = kOffXMl + (1 + kSoftmaxGroups) * kRows * 4;   // pair-count prefix [items + 1], then [item][4]: first row, rows, trajectory, length
constexpr int kOffUnits = kOffTable + (kMaxItems + 1) * 4 + kMaxItems * 16;   // ring of unit numbers
constexpr int kSmemUsed = kOffUnits + kUnitRing * 4;
constexpr int kSmemBytes = kSmemUsed + 1024;               // + slack for the 1024-byte alignment
static_assert(kSmemBytes <= 227 * 1024, "one block must fit an SM");
static_assert(kSoftmaxGroups < kSBufs, "a warpgroup finds the S of its next tile computed while it works on this one");

constexpr int kTmemCols = 512;             // S buffer b at columns b * 128; the tile's P (packed bf16) over its first 64 columns
constexpr int kTmemO = kSBufs * kKeys;     // O at 384
constexpr int kRedoBits = kChunkRedoBits;  // units of a launch are marked in a bitmap of this many bits (unit mod kRedoBits)

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
    uint32_t *redo_bits;        // kRedoBits bits, zero at launch: units whose rows outgrew the fixed reference max
    int *unit_counter;          // zero at launch: the next unit to hand out
    DeviceStatus *status;
};

// Bounded wait on a barrier of this CTA (its arrivals may come from the other CTA).  A wait that runs out raises the
// abort flag of both CTAs; from then on nobody in the pair waits, every role runs its bounded loops to the end.
template <bool kClusterScope = false>
__device__ __forceinline__ void pair_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t peer_abort,
                                          DeviceStatus *status, int where) {
    constexpr long long kWaitCycles = 2000000000LL;   // about a second
    auto poll = [&]() { return kClusterScope ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity); };
    if (poll()) return;
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (poll()) return;
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
    int *s_prefix = reinterpret_cast<int *>(smem + kOffTable);

    if (static_cast<int>(smem - smem_raw) + kSmemUsed > kSmemBytes) {   // cannot happen: the slack covers any alignment
        if (threadIdx.x == 0) report(prm.status, ROLLART_ERR_CUDA, static_cast<int>(smem - smem_raw), 3);
        return;
    }
    const uint32_t bars = smem_u32(smem + kOffBars);
    const uint32_t bar_qfull = bars, bar_qready = bars + 8u;
    // K(j) lives in stage j % kStagesK, V(j) in stage kStagesK + j % kStagesV; use u of a stage has parity u & 1
    auto stage_of = [&](int kv, int j) { return kv == 0 ? j % kStagesK : kStagesK + j % kStagesV; };
    auto use_of = [&](int kv, int j) { return kv == 0 ? j / kStagesK : j / kStagesV; };
    auto bar_full = [&](int s) { return bars + 8u * (2 + s); };                  // this CTA's copies have landed
    auto bar_empty = [&](int s) { return bars + 8u * (2 + kStages + s); };       // the MMAs that read the stage are done
    auto bar_ready = [&](int s) { return bars + 8u * (2 + 2 * kStages + s); };   // leader: both CTAs' halves are in place
    auto bar_sfull = [&](int b) { return bars + 8u * (2 + 3 * kStages + b); };
    auto bar_pfull = [&](int b) { return bars + 8u * (2 + 3 * kStages + kSBufs + b); };   // leader: P of both CTAs is stored in S buffer b
    const uint32_t bar_odone = bars + 8u * (2 + 3 * kStages + 2 * kSBufs);      // the last PV of a unit is done
    const uint32_t bar_qfree = bar_odone + 8u;                                   // the last QK of a unit is done: Q may be overwritten
    const uint32_t bar_ofree = bar_odone + 16u;                                  // leader: every softmax warp of the pair has read O
    auto bar_ufull = [&](int s) { return bar_odone + 8u * (3 + s); };             // ring slot s holds the next unit's number
    auto bar_uempty = [&](int s) { return bar_odone + 8u * (3 + kUnitRing + s); };   // second CTA: every role of the pair has read slot s
    const uint32_t peer_abort = map_to_cta(smem_u32(smem + kOffAbort), rank ^ 1u);

    // ---- set-up that does not depend on the unit, first: it overlaps the loads of the item table below ----
    // barriers (one per thread), Q zero fill (rows beyond tpt * g are never written by the copy), tensor memory
    const int v_warps = min(kVCopyWarps, max(1, kKeys / P / 2));   // V copy warps in use: at least two pages of a tile each
    const int k_warps = min(kKCopyWarps, max(1, kOwnKeys / P / 2));
    if (threadIdx.x < kNumBars) {
        const int i = static_cast<int>(threadIdx.x);
        uint32_t count = 1;                                                      // q_full, full, empty, s_full, o_done
        if (i == 1 || (i >= 2 + 2 * kStages && i < 2 + 3 * kStages)) count = 2;  // q_ready, ready: one arrival per CTA
        else if (i >= 2 && i < 2 + kStagesK) count = k_warps;                    // full of a K stage, likewise
        else if (i >= 2 + kStagesK && i < 2 + kStages) count = v_warps;          // full of a V stage: one arrival (with its bytes) per active V copy warp
        else if (i >= 2 + 3 * kStages + kSBufs && i < 2 + 3 * kStages + 2 * kSBufs) count = 8;   // p_full: 4 warps x 2 CTAs
        else if (i == 2 + 3 * kStages + 2 * kSBufs + 2) count = 8 * kSoftmaxGroups;   // o_free: every softmax warp of both CTAs
        else if (i >= kNumBars - kUnitRing) count = 2 * (kThreads / 32) - 1;     // unit_empty: every warp of the pair but the one that hands the units out
        mbar_init(bars + 8u * i, count);
    }
    if (threadIdx.x == 0) {
        *s_abort = 0;
        // an earlier block ran out of patience: the leader's reading of the flag decides for the pair
        s_fatal[0] = *reinterpret_cast<volatile int *>(&prm.status->fatal) != 0 ? 1 : 0;
    }
    for (int i = threadIdx.x; i < kTileQ / 16; i += kThreads) reinterpret_cast<uint4 *>(smem + kOffQ)[i] = make_uint4(0, 0, 0, 0);
    if (warp == 0) tmem_alloc_pair(smem_u32(smem + kOffTmemSlot), kTmemCols);

    // ---- the tables from which a unit number gives (item, kv head, pair of M-tiles): pairs per item -> prefix (searched
    //      per unit), and every item's rows, trajectory and length, so that a unit's geometry needs no (dependent)
    //      global loads ----
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
    const int total_units = s_prefix[prm.n_items] * hkv;
    // Units are numbered (item, head, pair) with the later (longer) pairs of an (item, head) first, and the persistent
    // pairs take them in that order, so the pairs re-reading the same keys run at the same time.  Every role walks the
    // same list of unit numbers and derives a unit's geometry from the tables by itself.
    struct Unit {
        bool active;
        int head, q_row0, n_chunk, t, L, prior, first_tok, toks, nmax, min_count;
    };
    auto unit_at = [&](int unit) {
        Unit u;
        int lo = 0, hi = prm.n_items;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_prefix[mid] * hkv <= unit) lo = mid; else hi = mid;
        }
        const int np = max(1, s_prefix[lo + 1] - s_prefix[lo]);
        const int rem = unit - s_prefix[lo] * hkv;
        u.head = rem / np;
        const int pair = np - 1 - (rem - u.head * np);      // later M-tiles see more keys: start the longest ones first
        u.q_row0 = s_item[4 * lo]; u.n_chunk = s_item[4 * lo + 1]; u.t = s_item[4 * lo + 2]; u.L = s_item[4 * lo + 3];
        int bad_value = 0;
        bool bad = false;
        if (u.q_row0 < 0 || u.n_chunk < 0 || static_cast<long long>(u.q_row0) + u.n_chunk > prm.total_q) { bad = true; bad_value = u.q_row0; }   // q_indptr does not describe rows of q
        else if (u.t < 0 || u.t >= prm.num_traj) { bad = true; bad_value = u.t; }
        else if (u.L < 0 || u.L > prm.max_seq_len || u.n_chunk > u.L) { bad = true; bad_value = u.L; }
        if (bad && warp == 1 && lane == 0 && rank == 0) report(prm.status, ROLLART_ERR_BOUNDS, bad_value, 3);
        u.active = !bad;                                      // a unit's state depends on the unit alone: every role of both CTAs decides alike
        if (bad) { u.L = 0; u.t = 0; }
        u.prior = u.L - u.n_chunk;
        u.first_tok = (2 * pair + static_cast<int>(rank)) * tpt;              // first chunk token of this CTA's M-tile
        u.toks = max(0, min(tpt, u.n_chunk - u.first_tok));                   // its live tokens (the second CTA may have none)
        const int pair_toks_end = min(u.n_chunk, (2 * pair + 2) * tpt);       // one past the pair's last live token
        u.nmax = (u.prior + pair_toks_end + kKeys - 1) / kKeys;               // key tiles of the pair (>= 1)
        u.min_count = min(u.L, u.prior + u.first_tok + 1);                    // keys the CTA's first row sees
        return u;
    };

    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();             // the zeroed Q rows are ordered before the copy that lands beside them
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();              // both CTAs' barriers exist before anything arrives on them
    tc_fence_after();
    const uint32_t tmem = *s_tmem;
    // (the leader stays resident until the pair's last common barrier, so its shared memory may be read here)
    const bool run = ld_cluster_u32(map_to_cta(smem_u32(smem + kOffFatal), 0)) == 0u;
    // The units of the launch are handed out in order from a counter in global memory, so a pair that finishes early
    // takes the next one (a fixed split left the slowest pair 2 % behind the mean, and more on a GPU whose SMs differ).
    // One warp of the second CTA (its MMA warp has nothing else to do) draws the numbers and puts each into a ring slot
    // of both CTAs; every other warp of the pair reads the slot and says so.  A negative number ends the walk.
    volatile int *s_units = reinterpret_cast<volatile int *>(smem + kOffUnits);
    const uint32_t giver_uempty = map_to_cta(bar_uempty(0), 1);
    auto next_unit = [&](int k) {
        const int slot = k % kUnitRing;
        pair_wait<true>(bar_ufull(slot), (k / kUnitRing) & 1, s_abort, peer_abort, prm.status, 16);
        const int unit = s_units[slot];
        __syncwarp();
        // (the arrival hangs on the value read, so the read is over before the slot can be written again; the arrival
        // itself needs no cluster-scope release, which would cost this warp ~1,100 cycles per unit)
        if (lane == 0 && unit >= -1) mbar_arrive_cluster(giver_uempty + 8u * slot);
        return *s_abort ? -1 : unit;
    };

    if (!run) {
        // fall through to the common exit
    } else if (warp < 4 || warp >= 12) {
      if (warp == 0 || warp == 3 || warp >= 12) {
        // =============================== copy warps ===============================
        // Warp 0 brings Q; warps 0 and 15 bring this CTA's 64 keys of every K tile (one box per page: its keys in
        // groups of 8, both 64-dim halves of a group side by side); warps 3 and 12..14 bring its 64 dims of every V tile
        // (one box per page, from the [rows][128 dims] view of the pool).  Each warp takes its share of a tile's pages.
        const int kv = (warp == 0 || warp == 15) ? 0 : 1;
        const int vpart = kv == 0 ? (warp == 15 ? 1 : 0) : (warp >= 12 ? warp - 11 : 0);   // which part of the tile's pages
        const int parts = kv == 0 ? k_warps : v_warps;
        const int pages_per_tile = kKeys / P;
        const int my_pages = (kv == 0 ? kOwnKeys / P : pages_per_tile) / parts;  // boxes this warp issues per tile
        const int my_first = (kv == 0 ? static_cast<int>(rank) * (kOwnKeys / P) : 0) + vpart * my_pages;   // first page of the tile it takes
        const int dst_first = vpart * my_pages;                                   // ... and where in the stage that page lands
        const int tiles_per_batch = 32 / pages_per_tile;
        const uint32_t box_bytes = static_cast<uint32_t>(P) * 128;                // P rows x 64 dims
        int gt = 0;                                                               // tiles copied so far, over all units: the ring position
        int nu = 0;                                                               // units taken so far
        for (int uk = 0;; ++uk) {
            const int unit = next_unit(uk);
            if (unit < 0) break;
            if (vpart >= parts) continue;                 // a copy warp that this page size leaves without pages
            const Unit u = unit_at(unit);
            if (!u.active) continue;
            if (warp == 0) {
                // Q of this unit, once the last QK of the unit before it has read the buffer
                if (nu > 0) pair_wait(bar_qfree, (nu - 1) & 1, s_abort, peer_abort, prm.status, 1);
                if (lane == 0) {
                    if (u.toks > 0) {
                        mbar_arrive_expect_tx(bar_qfull, static_cast<uint32_t>(tpt * g) * kRowBytes);
                        const uint32_t dst = smem_u32(smem + kOffQ);
                        tma_load_3d(dst, &qmap, bar_qfull, 0, u.head * g, u.q_row0 + u.first_tok);
                        tma_load_3d(dst + kHalfQ, &qmap, bar_qfull, 64, u.head * g, u.q_row0 + u.first_tok);
                    } else {
                        mbar_arrive(bar_qfull);      // no live row here: whatever Q holds, its rows are not written out
                    }
                }
                __syncwarp();
            }
            ++nu;
            const int32_t *table_row = prm.page_table + static_cast<long long>(u.t) * prm.max_pages;
            // Page ids are fetched 32 at a time, one per lane, and the next 32 are requested a whole batch ahead, so the
            // table lookup (a dependent load) is off the copy loop's path.
            auto load_ids = [&](int batch) {
                const int lp = batch * 32 + lane;
                int pg = -1;
                if (lp * P < u.L && lp < prm.max_pages) {
                    pg = __ldg(table_row + lp);
                    if (pg < 0 || pg >= prm.num_pages) {
                        if (warp == 3 && rank == 0) report(prm.status, ROLLART_ERR_BOUNDS, pg, 3);
                        pg = -1;
                    }
                }
                return pg;
            };
            int ids_cur = load_ids(0), ids_next = load_ids(1);
            for (int j = 0; j < u.nmax; ++j, ++gt) {
                const int within = j % tiles_per_batch;
                if (j > 0 && within == 0) {
                    if (*s_abort) break;
                    ids_cur = ids_next;
                    ids_next = load_ids(j / tiles_per_batch + 1);
                }
                int pg = __shfl_sync(0xffffffffu, ids_cur, (within * pages_per_tile + my_first + lane) & 31);
                if (lane >= my_pages) pg = -1;
                const uint32_t nvalid = __popc(__ballot_sync(0xffffffffu, pg >= 0));
                const int stage = stage_of(kv, gt);
                pair_wait(bar_empty(stage), (use_of(kv, gt) & 1) ^ 1, s_abort, peer_abort, prm.status, 1 + kv);
                if (lane == 0) mbar_arrive_expect_tx(bar_full(stage), nvalid * (kv == 0 ? 2u : 1u) * box_bytes);
                __syncwarp();
                if (pg >= 0) {
                    const uint32_t dst = smem_u32(smem + kOffKV + stage * kStageBytes) + (dst_first + lane) * (kv == 0 ? 2u : 1u) * box_bytes;
                    const int row = (pg * hkv + u.head) * P;
                    if (kv == 0) {
                        tma_load_4d(dst, &kmap, bar_full(stage), 0, 0, 0, row >> 3);   // both halves: 2 box_bytes per page
                    } else {
                        tma_load_2d(dst, &vmap, bar_full(stage), kOwnDims * static_cast<int>(rank), row);
                    }
                }
            }
        }
      } else if (warp == 2) {
        // =============================== stage warp ===============================
        // Waits for this CTA's copies of each ring slot and tells the leader.  In the last V tile the rows of keys at or
        // beyond L (dead slots of the last page, pages that were never copied) are zeroed first: their P is exactly 0,
        // but 0 x NaN would still poison O.
        const uint32_t leader_qready = map_to_cta(bar_qready, 0);
        int gt = 0, nu = 0;
        for (int uk = 0;; ++uk) {
            const int unit = next_unit(uk);
            if (unit < 0) break;
            const Unit u = unit_at(unit);
            if (!u.active) continue;
            pair_wait(bar_qfull, nu & 1, s_abort, peer_abort, prm.status, 5);
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_qready);
            ++nu;
            for (int r = 0; r < 2 * u.nmax; ++r) {       // K(0) V(0) K(1) V(1) ...: the order in which the copies were issued
                const int kv = r & 1, j = r >> 1;
                const int stage = stage_of(kv, gt + j);
                pair_wait(bar_full(stage), use_of(kv, gt + j) & 1, s_abort, peer_abort, prm.status, 6 + kv);
                const int key0 = j * kKeys;
                if (kv && key0 + kKeys > u.L) {
                    const uint32_t v_addr = smem_u32(smem + kOffKV + stage * kStageBytes);
                    const int first_dead = max(0, u.L - key0);
                    for (int idx = lane; idx < (kKeys - first_dead) * 8; idx += 32) {
                        const uint32_t a = v_addr + static_cast<uint32_t>(first_dead + (idx >> 3)) * 128u + static_cast<uint32_t>(idx & 7) * 16u;
                        asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0) : "memory");
                    }
                    fence_proxy_async();      // the zeroed rows become visible to the tensor core's reads
                }
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(bar_ready(stage), 0));
            }
            gt += u.nmax;
        }
      } else {
        // =============================== MMA warp (leader only) ===============================
        // Per unit one thread issues QK(0) QK(1) QK(2) | PV(j) QK(j+3) | ...: three S buffers, so S of the next two key
        // tiles is ready long before the softmax of this one ends.  MMAs run in issue order, which is what protects the
        // reuse of an S buffer (it holds P(j) until PV(j), issued before QK(j+3), has read it).
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
            int gt = 0, nu = 0;                        // key tiles and units so far: ring positions and barrier phases run on
            auto issue_qk = [&](int j, bool last_of_unit) {   // j counts tiles over all units
                const int stage = stage_of(0, j);
                pair_wait(bar_ready(stage), use_of(0, j) & 1, s_abort, peer_abort, prm.status, 8);   // K(j), both halves
                tc_fence_after();
                const uint64_t k_desc = smem_desc(kv_addr + stage * kStageBytes, 16, 2048);   // 8-key groups 2 KB apart
                const uint32_t s_tm = tm + (j % kSBufs) * kKeys;
#pragma unroll
                for (int ks = 0; ks < kHeadDim / 16; ++ks) {   // 16 dims per step; the second 64 dims live in the other half
                    const uint64_t qoff = static_cast<uint64_t>(((ks >> 2) * kHalfQ + (ks & 3) * 32) >> 4);
                    const uint64_t koff = static_cast<uint64_t>(((ks >> 2) * 1024 + (ks & 3) * 32) >> 4);
                    if (elected) umma_pair_bf16(s_tm, q_desc + qoff, k_desc + koff, kIdescQK, ks > 0 ? 1u : 0u);
                }
                if (elected) {
                    umma_pair_commit(bar_sfull(j % kSBufs));
                    umma_pair_commit(bar_empty(stage));
                    if (last_of_unit) umma_pair_commit(bar_qfree);      // Q of the next unit may land
                }
                __syncwarp();
            };
            for (int uk = 0;; ++uk) {
                const int unit = next_unit(uk);
                if (unit < 0) break;
                const Unit u = unit_at(unit);
                if (!u.active) continue;
                const int nmax = u.nmax;
                pair_wait(bar_qready, nu & 1, s_abort, peer_abort, prm.status, 9);
                for (int j = 0; j < kSBufs && j < nmax; ++j) issue_qk(gt + j, j == nmax - 1);
                for (int j = 0; j < nmax; ++j) {
                    const int stage = stage_of(1, gt + j), sb = (gt + j) % kSBufs;
                    pair_wait(bar_ready(stage), use_of(1, gt + j) & 1, s_abort, peer_abort, prm.status, 10);   // V(j), both halves
                    // V half tile is [key][128 B]: the 16 keys of step ks start 2 KB further on; 8-key groups are 1 KB apart
                    const uint64_t v_desc = smem_desc(kv_addr + stage * kStageBytes, 1024);
                    const uint32_t p_tm = tm + sb * kKeys;
                    pair_wait(bar_pfull(sb), ((gt + j) / kSBufs) & 1, s_abort, peer_abort, prm.status, 11);
                    // the first PV of a unit overwrites O: every softmax warp of the pair has read the unit before by then
                    if (j == 0 && nu > 0) pair_wait(bar_ofree, (nu - 1) & 1, s_abort, peer_abort, prm.status, 15);
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < kKeys / 16; ++ks)       // 16 keys per step: 8 packed columns of P's row
                        if (elected)
                            umma_pair_bf16_ts(tm + kTmemO, p_tm + ks * 8, v_desc + static_cast<uint64_t>((ks * 16 * 128) >> 4), kIdescPV,
                                              (j > 0 || ks > 0) ? 1u : 0u);
                    __syncwarp();
                    if (elected) {
                        umma_pair_commit(bar_empty(stage));
                        if (j == nmax - 1) umma_pair_commit(bar_odone);
                    }
                    __syncwarp();
                    if (j + kSBufs < nmax) issue_qk(gt + j + kSBufs, j + kSBufs == nmax - 1);
                }
                gt += nmax;
                ++nu;
            }
        }
        else {
            // =============================== the second CTA's warp 1 hands out the units ===============================
            const uint32_t leader_units = map_to_cta(smem_u32(smem + kOffUnits), 0), leader_ufull = map_to_cta(bar_ufull(0), 0);
            const uint32_t own_ufull = map_to_cta(bar_ufull(0), 1);
            for (int k = 0;; ++k) {
                const int slot = k % kUnitRing;
                if (k >= kUnitRing) pair_wait<true>(bar_uempty(slot), (k / kUnitRing - 1) & 1, s_abort, peer_abort, prm.status, 17);
                int unit = 0;
                if (lane == 0) {
                    unit = atomicAdd(prm.unit_counter, 1);
                    if (unit >= total_units || *s_abort) unit = -1;
                    s_units[slot] = unit;
                    st_cluster_u32(leader_units + 4u * slot, static_cast<uint32_t>(unit));
                    mbar_arrive_cluster_release(leader_ufull + 8u * slot);
                    mbar_arrive_cluster_release(own_ufull + 8u * slot);
                }
                unit = __shfl_sync(0xffffffffu, unit, 0);
                if (unit < 0) break;
            }
        }
        __syncwarp();
      }
    } else {
        // =============================== softmax warpgroups ===============================
        // Warpgroup w takes the key tiles j = w, w + 2, ...: one thread per query row takes all 128 scores of the row.
        // The two warps of an SM sub-partition work on different tiles, so each one's waits (for S, for tensor-memory
        // loads and stores) fall into the arithmetic of the other.
        const int wg = (warp - 4) >> 2;
        const int quarter = warp & 3;                         // tensor-memory lanes 32 * quarter .. + 31 belong to this warp
        const int row = quarter * 32 + lane;
        const uint32_t lane_addr = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        const int tok_local = row / g, head_local = row - tok_local * g;
        const float scale = prm.scale_log2;
        const uint32_t leader_pfull = map_to_cta(bar_pfull(0), 0);
        const uint32_t leader_ofree = map_to_cta(bar_ofree, 0);
        volatile float *x_m = reinterpret_cast<volatile float *>(smem + kOffXMl);   // [row]
        volatile float *x_l = x_m + kRows;                                            // [warpgroup][row]
        uint32_t sa[32], sb[32];            // two quarters (32 columns each) of the row's scores
        int gt = 0, nu = 0;                 // key tiles and units so far: S buffers and barrier phases run on over the units

      for (int uk = 0;; ++uk) {
        const int unit = next_unit(uk);
        if (unit < 0) break;
        const Unit u = unit_at(unit);
        if (!u.active) continue;
        const int nmax = u.nmax, min_count = u.min_count;
        const bool live = tok_local < u.toks;
        const int count = min(u.L, u.prior + u.first_tok + min(tok_local, max(u.toks, 1) - 1) + 1);   // keys this row sees (>= 1)
        float l_sum = 0.f;
        bool outgrown = false;
        int poly_top = INT_MIN;             // the largest argument handed to the FMA-pipe exponential (see ex2_poly2)

        // ---- the row's reference max: the largest visible score of the first tile (every row sees key 0) ----
        if (wg == 0) {
            pair_wait(bar_sfull(gt % kSBufs), (gt / kSBufs) & 1, s_abort, peer_abort, prm.status, 12);
            tc_fence_after();
            const bool need_mask = kKeys > min_count;
            float rmax = -INFINITY;
            auto quarter_max = [&](const uint32_t (&r)[32], int col0) {
                if (!need_mask) {
                    // the max of scale * s is scale * (max or min of s): the extreme of the raw scores by 3-input ops
                    float e[4];
                    if (scale >= 0.f) {
#pragma unroll
                        for (int k = 0; k < 4; ++k) e[k] = max3(__uint_as_float(r[k]), __uint_as_float(r[4 + k]), __uint_as_float(r[8 + k]));
#pragma unroll
                        for (int k = 0; k < 4; ++k) e[k] = max3(e[k], __uint_as_float(r[12 + k]), __uint_as_float(r[16 + k]));
#pragma unroll
                        for (int k = 0; k < 4; ++k) e[k] = max3(e[k], __uint_as_float(r[20 + k]), __uint_as_float(r[24 + k]));
#pragma unroll
                        for (int k = 0; k < 4; ++k) e[k] = fmaxf(e[k], __uint_as_float(r[28 + k]));
                        rmax = fmaxf(rmax, fmaxf(fmaxf(e[0], e[1]), fmaxf(e[2], e[3])) * scale);
                    } else {
#pragma unroll
                        for (int k = 0; k < 4; ++k) e[k] = min3(__uint_as_float(r[k]), __uint_as_float(r[4 + k]), __uint_as_float(r[8 + k]));
#pragma unroll
                        for (int k = 0; k < 4; ++k) e[k] = min3(e[k], __uint_as_float(r[12 + k]), __uint_as_float(r[16 + k]));
#pragma unroll
                        for (int k = 0; k < 4; ++k) e[k] = min3(e[k], __uint_as_float(r[20 + k]), __uint_as_float(r[24 + k]));
#pragma unroll
                        for (int k = 0; k < 4; ++k) e[k] = fminf(e[k], __uint_as_float(r[28 + k]));
                        rmax = fmaxf(rmax, fminf(fminf(e[0], e[1]), fminf(e[2], e[3])) * scale);
                    }
                } else {
                    // masked tile: keys the row does not see are left out (their scores may be anything)
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (col0 + c < count) rmax = fmaxf(rmax, __uint_as_float(r[c]) * scale);
                }
            };
            const uint32_t s_addr = lane_addr + (gt % kSBufs) * kKeys;   // the unit's first tile
            tmem_ld32(s_addr, sa);
            tmem_ld32(s_addr + 32, sb);
            tmem_wait_ld_of(sa);
            tmem_wait_ld_of(sb);
            quarter_max(sa, 0);
            quarter_max(sb, 32);
            tmem_ld32(s_addr + 64, sa);
            tmem_ld32(s_addr + 96, sb);
            tmem_wait_ld_of(sa);
            tmem_wait_ld_of(sb);
            quarter_max(sa, 64);
            quarter_max(sb, 96);
            x_m[row] = rmax;
            // (a reference of -inf, +inf or NaN, i.e. scores that are not finite, ends in a row sum that marks the unit)
        }
        named_bar_sync(1, 128 * kSoftmaxGroups);              // the other warpgroup takes the reference from here
        const float neg_m = -x_m[row];

        for (int j = wg; j < nmax; j += kSoftmaxGroups) {
            const int sbuf = (gt + j) % kSBufs;
            const uint32_t s_addr = lane_addr + sbuf * kKeys;
            pair_wait(bar_sfull(sbuf), ((gt + j) / kSBufs) & 1, s_abort, peer_abort, prm.status, 12);
            tc_fence_after();
            const int key0 = j * kKeys;
            const bool need_mask = key0 + kKeys > min_count;    // the same for every thread of the CTA
            const int live_keys = count - key0;                 // of this tile's 128 keys, those the row sees
            float rs[4] = {0.f, 0.f, 0.f, 0.f};
            // P = exp2(scale * s - m) for 32 keys of the row (quarter q of the tile), packed to bf16: 16 columns at
            // the start of the S buffer, which the scores of quarter q have left by then.  Two copies of the pass,
            // chosen once per tile: the unmasked one carries no compare / select.  One pair of exponentials in
            // kPolyOneIn goes to the FMA pipe.
            auto exp_pass = [&](auto masked_tag, auto q_tag, const uint32_t (&r)[32]) {
                constexpr bool kMasked = decltype(masked_tag)::value;
                constexpr int q = decltype(q_tag)::value;
                uint32_t packed[16];
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                    float x0, x1, p0, p1;
                    fma2(x0, x1, __uint_as_float(r[c]), __uint_as_float(r[c + 1]), scale, neg_m);
                    if (((q * 16 + (c >> 1)) % kPolyOneIn) == kPolyOneIn - 1) {
                        ex2_poly2(p0, p1, x0, x1, poly_top);
                    } else {
                        p0 = ex2(x0);
                        p1 = ex2(x1);
                    }
                    if constexpr (kMasked) {
                        p0 = q * 32 + c < live_keys ? p0 : 0.f;
                        p1 = q * 32 + c + 1 < live_keys ? p1 : 0.f;
                    }
                    add2(rs[c & 2], rs[(c & 2) + 1], p0, p1);
                    packed[c >> 1] = pack_bf16(p0, p1);
                }
                tmem_st16(s_addr + q * 16, packed);      // P as the next A operand
            };
            auto pass = [&](auto q_tag, const uint32_t (&r)[32]) {
                if (need_mask) exp_pass(std::true_type{}, q_tag, r); else exp_pass(std::false_type{}, q_tag, r);
            };
            // each load stays in flight behind the arithmetic of the quarter before it
            tmem_ld32(s_addr, sa);
            tmem_ld32(s_addr + 32, sb);
            tmem_wait_ld_of(sa);
            tmem_wait_ld_of(sb);
            pass(std::integral_constant<int, 0>{}, sa);
            tmem_ld32(s_addr + 64, sa);
            pass(std::integral_constant<int, 1>{}, sb);
            tmem_wait_ld_of(sa);
            tmem_ld32(s_addr + 96, sb);
            pass(std::integral_constant<int, 2>{}, sa);
            tmem_wait_ld_of(sb);
            pass(std::integral_constant<int, 3>{}, sb);
            const float rsum = (rs[0] + rs[1]) + (rs[2] + rs[3]);
            outgrown = outgrown || !(rsum <= kRowSumLimit);       // also true for inf / NaN
            l_sum += rsum;
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_pfull + 8u * sbuf);
        }

        // a row that outgrew its reference (or whose scores are not finite): the unit is computed again by the kernel
        // that moves the reference max
        outgrown = live && (outgrown || poly_top > kPolyArgTop);
        if (__any_sync(0xffffffffu, outgrown) && lane == 0)
            atomicOr(prm.redo_bits + ((unit % kRedoBits) >> 5), 1u << (unit & 31));

        // ---- epilogue: O / l -> bf16 rows of out; warpgroup w writes dims 64 w .. 64 w + 63 ----
        x_l[wg * kRows + row] = l_sum;
        named_bar_sync(1, 128 * kSoftmaxGroups);
        {
            pair_wait(bar_odone, nu & 1, s_abort, peer_abort, prm.status, 14);
            tc_fence_after();
            const float l_all = x_l[row] + x_l[kRows + row];
            const float inv = l_all > 0.f ? prm.out_scale / l_all : 0.f;
            const uint32_t o_addr = lane_addr + kTmemO + wg * 64;
            const long long orow = (static_cast<long long>(u.q_row0 + u.first_tok + tok_local) * prm.num_q_heads + u.head * g + head_local);
#pragma unroll 1
            for (int c0 = 0; c0 < 64; c0 += 32) {
                tmem_ld32(o_addr + c0, sa);
                tmem_wait_ld_of(sa);
                if (live) {
                    uint4 *dst = reinterpret_cast<uint4 *>(prm.out + orow * kHeadDim + wg * 64 + c0);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        uint4 v;
                        v.x = pack_bf16(__uint_as_float(sa[8 * k]) * inv, __uint_as_float(sa[8 * k + 1]) * inv);
                        v.y = pack_bf16(__uint_as_float(sa[8 * k + 2]) * inv, __uint_as_float(sa[8 * k + 3]) * inv);
                        v.z = pack_bf16(__uint_as_float(sa[8 * k + 4]) * inv, __uint_as_float(sa[8 * k + 5]) * inv);
                        v.w = pack_bf16(__uint_as_float(sa[8 * k + 6]) * inv, __uint_as_float(sa[8 * k + 7]) * inv);
                        dst[k] = v;
                    }
                }
            }
            if (live && wg == 0 && prm.lse != nullptr) prm.lse[orow] = l_all > 0.f ? (-neg_m + log2f(l_all)) * kLn2 : -INFINITY;
            // O has been read: the first PV of the pair's next unit may overwrite it
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_ofree);
        }
        gt += nmax;
        ++nu;
      }
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

cudaError_t launch_chunk_attn_pair(const AttnCall &c, int base, int n, cudaStream_t stream, int64_t *launches) {
    const int hkv = c.pool.num_kv_heads, g = c.num_q_heads / hkv, tpt = kRows / g;
    cudaError_t e = cudaFuncSetAttribute(chunk_attn_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    CUtensorMap qmap, kmap, vmap;
    if (!encode_q_map(&qmap, c.q, c.total_q, c.num_q_heads, g) ||
        !encode_pool_groups(&kmap, c.pool.k, c.pool.num_pages, hkv, c.pool.page_size) ||
        !encode_pool_rows(&vmap, c.pool.v, c.pool.num_pages, hkv, c.pool.page_size))
        return cudaErrorInvalidValue;
    PairParams prm;
    prm.page_table = c.trajs.page_table; prm.seq_lens = c.trajs.seq_lens;
    prm.traj_ids = c.traj_ids ? c.traj_ids + base : nullptr;
    prm.q_indptr = c.q_indptr + base;
    prm.max_pages = c.trajs.max_pages; prm.num_traj = c.trajs.num_traj; prm.num_pages = c.pool.num_pages;
    prm.page_size = c.pool.page_size; prm.num_kv_heads = hkv; prm.num_q_heads = c.num_q_heads; prm.group = g;
    prm.n_items = n; prm.item_offset = base; prm.max_seq_len = c.max_seq_len; prm.total_q = c.total_q;
    prm.out = c.out; prm.lse = c.lse; prm.scale_log2 = c.sm_scale * kLog2e; prm.out_scale = c.v_scale;
    prm.redo_bits = c.redo_bits; prm.unit_counter = reinterpret_cast<int *>(c.redo_bits + kRedoBits / 32); prm.status = c.status;
    // an upper bound on the M-tile pairs of these items: every item has at most one ragged pair
    const long long pairs = (static_cast<long long>(c.total_q) + 2 * tpt - 1) / (2 * tpt) + n;
    if (pairs * hkv > 0x3FFFFFFFLL) return cudaErrorInvalidValue;
    // persistent pairs: one cluster per two SMs (or fewer, when there are fewer units), taking the units from the counter
    const long long clusters = std::max(1LL, std::min<long long>(pairs * hkv, (c.sm_count > 1 ? c.sm_count : 2) / 2));
    chunk_attn_pair_kernel<<<static_cast<unsigned>(2 * clusters), kThreads, kSmemBytes, stream>>>(qmap, kmap, vmap, prm);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace rollart
