// The staged sweep: one persistent kernel that plans, streams and merges.
//
// Section 5 of the Q-First paper lets a cache be split anywhere: partial states
// (W, Z) add over disjoint token sets.  The user-visible split is the shard; this
// kernel splits further, invisibly, so that every SM streams the same number of KV
// bytes whatever the batch looks like.
//
//   plan      every CTA turns (seq_lens, shard_ranges) into a prefix sum over "stage
//             units" (8 pages = 128 tokens of one KV head of one shard) in shared
//             memory.  The unit space is cut into pieces (PieceGrid): one equal static
//             slice per CTA over the first nine tenths, and chunks of halving size over
//             the rest, which CTAs draw from a counter as they run out of work.  Batches
//             with more than kMaxSmemEntries (request, shard) pairs use a separate plan
//             kernel that leaves the prefix in scratch (and static slices only).
//   stream    a producer warp walks its pieces, looks pages up in the block table and
//             issues one 4 KB TMA box per K or V page (128B-swizzled) into a 3-stage shared-memory ring;
//             8 consumer warps each take one page of a stage: S = K Q^T on tensor cores
//             (tokens on M, the group's heads on N), fp32 online softmax, P split into
//             bf16 hi+lo, O^T += V^T P^T.
//   merge     at a segment end the eight warps' states merge through shared memory into
//             the shard's state, or, if a piece boundary cut the (shard, KV head) unit,
//             into a segment slot of the scratch that the finish kernel (qf_finish.cuh)
//             merges after the sweep.  Empty shards get (0, -inf, -inf) from the consumer
//             warps' prologue.
//
// All waits are bounded: a wait that runs out sets QF_STATUS_TIMEOUT, raises a
// CTA-wide abort flag and every warp leaves.  No CTA ever waits for another CTA
// (drawing a chunk is one atomic add; it never blocks on another CTA's progress).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdio>
#include <chrono>
#include <mutex>

#include "qf_common.cuh"
#include "qf_page_math.cuh"
#include "qf_finish.cuh"

namespace qf {

constexpr int kConsumerWarps = 8;
constexpr int kPagesPerStage = kConsumerWarps;    // pages (of one KV head) per ring stage, one per consumer warp
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kSweepThreads  = (kConsumerWarps + 1) * 32;
constexpr int kStages        = 3;                 // 3 x 64 KB of K and V in flight per SM
constexpr int kMaxSweepCtas  = 160;               // persistent CTAs (one per SM) are capped at this
constexpr int kHalfTileBytes = 2048;              // 16 rows x 64 channels of bf16
constexpr int kRedStride     = kHeadDim + 4;      // padded row of the warp-merge buffer
constexpr int kMaxSmemEntries = 2048;             // (request, shard) pairs planned in shared memory
// Tail balancing of the unit kernel: the last 1/kDynDivisor of the stage-unit space is cut into chunks that
// the CTAs draw from a counter as they run out of work (see PieceGrid).
#ifndef QF_DYN_DIVISOR
#define QF_DYN_DIVISOR 10
#endif
#ifndef QF_DYN_MIN_CHUNK
#define QF_DYN_MIN_CHUNK 3
#endif
constexpr int kDynDivisor       = QF_DYN_DIVISOR;
constexpr int kDynMinChunk      = QF_DYN_MIN_CHUNK;   // stage units
#ifndef QF_DYN_ROUNDS
#define QF_DYN_ROUNDS 3
#endif
constexpr int kDynRounds        = QF_DYN_ROUNDS;      // chunk sizes halve from round to round
constexpr int kMaxDynChunks     = kDynRounds * kMaxSweepCtas;   // bounds the segment slots
constexpr int kDynMinUnitsPerCta = 112;               // shorter sweeps (under ~150 us) stay fully static: measured break-even
static_assert(kMaxSweepCtas + kMaxDynChunks < (1 << kEpochShift), "segments of one unit must fit the arrival count");

struct WorkspaceLayout {
    size_t header_off, prefix_off, counter_off, piece_off, seg_off, total;
    size_t seg_slots;
    int seg_stride;  // floats per segment slot
};

inline int seg_stride_floats(int G) { return G * kHeadDim + ((2 * G + 3) & ~3); }

inline WorkspaceLayout workspace_layout(int batch, int max_shards, int num_kv_heads, int G)
{
    WorkspaceLayout L;
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t entries = (size_t)batch * max_shards;
    L.header_off = 0;
    L.prefix_off = 256;
    L.counter_off = up(L.prefix_off + (entries + 1) * sizeof(int));
    L.piece_off = up(L.counter_off + entries * num_kv_heads * sizeof(unsigned long long));
    L.seg_off = up(L.piece_off + (size_t)(kMaxSweepCtas + kMaxDynChunks) * sizeof(int4));
    L.seg_stride = seg_stride_floats(G);
    // a cut unit's segment lives in slot (unit + piece): both grow along the unit space, so slots are unique
    const size_t slots = entries * num_kv_heads + (size_t)kMaxSweepCtas + (size_t)kMaxDynChunks;
    L.seg_slots = slots;
    L.total = up(L.seg_off + slots * L.seg_stride * sizeof(float));
    return L;
}

// Work units of entry e = (request, shard), all KV heads together: stage units of kPagesPerStage pages
// per KV head.
__device__ __forceinline__ int entry_units(const int *__restrict__ seq_lens, const int *__restrict__ shard_ranges,
                                           int e, int max_shards, int num_kv_heads, int max_tokens)
{
    int beg, end;
    clamp_range(shard_ranges[2 * e], shard_ranges[2 * e + 1], seq_lens[e / max_shards], max_tokens, beg, end);
    if (end <= beg) return 0;
    const int npages = ((end - 1) >> 4) - (beg >> 4) + 1;
    return ((npages + kPagesPerStage - 1) / kPagesPerStage) * num_kv_heads;
}

// The stage-unit space [0, total) is cut into pieces, each swept by one CTA front to back.  Pieces
// 0..n_ctas-1 are equal static slices of [0, static_end): CTA c starts with piece c.  The rest, when the
// sweep is long enough to pay for it, is cut into chunks that CTAs draw from a counter when they run out
// of work: SMs do not stream at the same rate (a few percent, stable per SM), and with static slices alone
// the slowest SM sets the kernel's time.  Chunks come in kDynRounds rounds of at most n_ctas chunks; every
// round but the last takes half of what is left, so chunk sizes halve and a chunk is never more than a
// 1/n_ctas share of the work still to be drawn when it is drawn; the kernel's end is then uneven by about
// one chunk of the last round.  The grid of pieces depends only on (total, n_ctas), never on who draws
// what, so a unit's segments and their merge order are fixed.
struct PieceGrid {
    int slice;        // units per static slice (>= 1)
    int static_end;   // units covered by static slices
    int n_chunks;
    int r_start[kDynRounds + 1];   // first unit of round r (r_start[kDynRounds] = total)
    int r_first[kDynRounds + 1];   // first chunk of round r
    int r_size[kDynRounds];        // units per chunk in round r (the round's last chunk may be shorter)
};
__host__ __device__ __forceinline__ int imin(int a, int b) { return a < b ? a : b; }
__host__ __device__ __forceinline__ int imax(int a, int b) { return a > b ? a : b; }
__host__ __device__ __forceinline__ PieceGrid piece_grid(int total, int n_ctas, bool allow_dynamic, bool always)
{
    PieceGrid g;
    const int min_total = always ? 2 * n_ctas : n_ctas * kDynMinUnitsPerCta;   // static slices of at least one unit
    if (!allow_dynamic || total < min_total) {
        g.slice = imax(1, (total + n_ctas - 1) / n_ctas);
        g.static_end = total;
    } else {
        g.slice = (total - total / kDynDivisor) / n_ctas;
        g.static_end = g.slice * n_ctas;
    }
    int off = g.static_end, idx = 0;
#pragma unroll
    for (int r = 0; r < kDynRounds; ++r) {
        const int rem = total - off;
        const int share = (r == kDynRounds - 1) ? rem : (rem + 1) / 2;
        const int size = imax(kDynMinChunk, (share + n_ctas - 1) / n_ctas);
        g.r_start[r] = off;
        g.r_first[r] = idx;
        g.r_size[r] = size;
        off += share;
        idx += (share + size - 1) / size;
    }
    g.r_start[kDynRounds] = total;
    g.r_first[kDynRounds] = idx;
    g.n_chunks = idx;
    return g;
}
__host__ __device__ __forceinline__ int piece_of(const PieceGrid &g, int n_ctas, int pos)
{
    if (pos < g.static_end) return pos / g.slice;
    int piece = 0;
#pragma unroll
    for (int r = 0; r < kDynRounds; ++r)
        if (pos >= g.r_start[r] && pos < g.r_start[r + 1]) piece = n_ctas + g.r_first[r] + (pos - g.r_start[r]) / g.r_size[r];
    return piece;
}
__host__ __device__ __forceinline__ void piece_range(const PieceGrid &g, int n_ctas, int piece, int &pos0, int &pos1)
{
    if (piece < n_ctas) {
        const long long lo = (long long)piece * g.slice, hi = lo + g.slice;
        pos0 = lo < g.static_end ? (int)lo : g.static_end;
        pos1 = hi < g.static_end ? (int)hi : g.static_end;
        return;
    }
    const int k = piece - n_ctas;
    pos0 = pos1 = g.r_start[kDynRounds];
#pragma unroll
    for (int r = 0; r < kDynRounds; ++r)
        if (k >= g.r_first[r] && k < g.r_first[r + 1]) {
            pos0 = g.r_start[r] + (k - g.r_first[r]) * g.r_size[r];
            pos1 = imin(pos0 + g.r_size[r], g.r_start[r + 1]);
        }
}

// ------------------------------------------------------------------ plan kernel (large batches only)
// prefix[e] = number of stage units before entry e = b*S + s, left in scratch.
__global__ void __launch_bounds__(1024)
plan_kernel(const int *__restrict__ seq_lens, const int *__restrict__ shard_ranges, int *__restrict__ prefix,
            int n_entries, int max_shards, int num_kv_heads, int max_tokens)
{
    __shared__ int warp_sums[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int carry = 0;
    for (int base = 0; base < n_entries; base += 1024) {
        const int e = base + tid;
        const int cnt = (e < n_entries) ? entry_units(seq_lens, shard_ranges, e, max_shards, num_kv_heads, max_tokens) : 0;
        int x = cnt;  // inclusive scan within the warp
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, x, off);
            if (lane >= off) x += y;
        }
        if (lane == 31) warp_sums[warp] = x;
        __syncthreads();
        int before = 0, chunk = 0;
        for (int w = 0; w < 32; ++w) {
            const int v = warp_sums[w];
            if (w < warp) before += v;
            chunk += v;
        }
        if (e < n_entries) prefix[e] = carry + before + x - cnt;
        carry += chunk;
        __syncthreads();
    }
    if (tid == 0) prefix[n_entries] = carry;
}

// ------------------------------------------------------------------ sweep kernel
struct __align__(16) StageMeta {
    int entry;     // b*S + s; -1 = no more work
    int kv_head;
    int page0;     // first logical page of this stage
    int npages;    // 1..8
    int tok_beg;   // clamped shard range
    int tok_end;
    int flags;     // bit0 first stage of a segment, bit1 last stage; bits 8..: segments the unit is cut into
    int aux;       // bits 0..7: pages whose table entry was out of range
    int slot;      // this segment's slot: the unit's first slot + the segment's ordinal (used when the unit is cut)
    int pad[3];
};
enum { kSegFirst = 1, kSegLast = 2 };

template <int G>
struct SweepSmem {
    // every K/V half tile is a 1024-byte-aligned 128B-swizzled TMA destination
    alignas(1024) uint8_t kv[kStages][2][kPagesPerStage][kPageBytes];  // [stage][K|V][page][half][row][128B]
    alignas(16) uint16_t q[kStages][G * kHeadDim];
    static constexpr int kRoundHeads = G < 4 ? G : 4;  // heads merged per epilogue round
    alignas(16) float red_acc[kConsumerWarps][kRoundHeads][kRedStride];
    alignas(16) float red_ml[kConsumerWarps][G][2];
    alignas(16) StageMeta meta[kStages];
    alignas(8) unsigned long long full_bar[kStages];
    alignas(8) unsigned long long empty_bar[kStages];
    alignas(8) unsigned long long red_bar[2];
    int abort_flag;
    unsigned long long epoch;   // this launch's epoch, read once per CTA
    int scan_ws[kConsumerWarps + 1];
    int prefix[kMaxSmemEntries + 1];
};

template <int G>
__global__ void __launch_bounds__(kSweepThreads, 1)
sweep_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
             const uint16_t *__restrict__ q, const int *__restrict__ block_table,
             const int *__restrict__ seq_lens, const int *__restrict__ shard_ranges,
             float *__restrict__ o_part, float *__restrict__ m_part, float *__restrict__ lse_part,
             unsigned long long *__restrict__ header, const int *__restrict__ global_prefix,
             int4 *__restrict__ piece_info, float *__restrict__ seg, int seg_stride,
             unsigned long long host_epoch, DevParams P)
{
    extern __shared__ uint8_t smem_raw[];
    SweepSmem<G> &sm = *reinterpret_cast<SweepSmem<G> *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int S = P.max_shards, Hkv = P.num_kv_heads, Hq = P.num_q_heads;
    const int n_entries = P.batch * S;
    const int max_tokens = P.max_tokens;
    volatile int *abort_flag = &sm.abort_flag;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&sm.full_bar[s]), 1);
            mbar_init(smem_u32(&sm.empty_bar[s]), kConsumerWarps);
        }
        mbar_init(smem_u32(&sm.red_bar[0]), kConsumerWarps);
        mbar_init(smem_u32(&sm.red_bar[1]), kConsumerWarps);
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    grid_dependency_wait();     // nothing above touches global memory
    grid_launch_dependents();
    if (tid == kConsumerThreads) {
        // the producer warp's first lane is idle during the plan below: it fetches the launch's epoch
        const unsigned long long ep = launch_epoch(header, host_epoch);
        sm.epoch = ep;
        if (blockIdx.x == 0) header[kHdrLastEpoch] = ep;
    }

    // ---- plan: prefix sum over (request, shard) entries, in shared memory when it fits
    const int *prefix;
    if (global_prefix) {
        prefix = global_prefix;
        __syncthreads();
    } else {
        int carry = 0;
        for (int base = 0; base < n_entries; base += kConsumerThreads) {
            const int e = base + tid;
            const int cnt = (tid < kConsumerThreads && e < n_entries)
                                ? entry_units(seq_lens, shard_ranges, e, S, Hkv, max_tokens) : 0;
            int x = cnt;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, x, off);
                if (lane >= off) x += y;
            }
            if (lane == 31) sm.scan_ws[warp] = x;
            __syncthreads();
            int before = 0, chunk = 0;
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) {
                const int v = sm.scan_ws[w];
                if (w < warp) before += v;
                chunk += v;
            }
            if (tid < kConsumerThreads && e < n_entries) sm.prefix[e] = carry + before + x - cnt;
            carry += chunk;
            __syncthreads();
        }
        if (tid == 0) sm.prefix[n_entries] = carry;
        __syncthreads();
        prefix = sm.prefix;
    }
    const unsigned long long epoch = sm.epoch;   // written before the plan's barriers
    if (P.check_bounds && blockIdx.x == 0) {
        // a cached length that the request's block-table row cannot address was clamped by the plan: report it
        for (int b = tid; b < P.batch; b += kSweepThreads)
            if (seq_lens[b] > max_tokens) epoch_or(header + kHdrStatus, epoch, kStatusBadPage);
    }
    const int total = prefix[n_entries];
    const int n_ctas = (int)gridDim.x;
    // a prefix left in global memory (very large batches) makes locating a piece's first entry slow: static only
    const PieceGrid pg = piece_grid(total, n_ctas, global_prefix == nullptr, P.draw_always != 0);
    if (blockIdx.x == 0 && tid == 0)
        header[kHdrTotals] = (unsigned long long)(unsigned)total | ((unsigned long long)(unsigned)(n_ctas + pg.n_chunks) << 32);

    if (warp == kConsumerWarps) {
        // ============================ producer warp ============================
        const unsigned long long kv_policy = l2_evict_first_policy();
        // the chunk counter must carry this launch's tag before this CTA draws from it (two round trips to L2 that
        // sweeps without a drawn tail, the short ones, do not pay)
        if (pg.n_chunks > 0 && lane == 0) epoch_counter_open(header + kHdrChunk, epoch);
        int stage = 0;
        uint32_t phase = 0;
        int issued = 0;
        bool ok = true;
        int piece = (int)blockIdx.x;
        int e = 0;
        // Per-segment metadata is kept off the critical path: a shard's token range and the first batch
        // of its block-table row are the same for all KV heads of the shard, so they are cached in
        // registers; the next non-empty shard's are fetched one segment ahead.
        int cur_e = -1, beg = 0, end = 0;
        int nxt_e = -1, nxt_r0 = 0, nxt_r1 = 0, nxt_len = 0;   // raw range of the next non-empty shard
        int head_tbl_e = -1, head_tbl = 0;                     // table entries of pages [first_page, +32) of a shard
        int nxt_tbl_e = -1, nxt_tbl = 0;
        auto load_tbl = [&](int b_, int page0_, int last_page_) -> int {
            const long long rb = (long long)b_ * P.max_pages_per_req;
            const int lp = min(page0_ + lane, last_page_);
            return block_table ? block_table[rb + lp] : (int)(rb + lp);
        };
        for (;;) {   // pieces: the static slice, then chunks drawn from the counter
            int pos, pos1;
            piece_range(pg, n_ctas, piece, pos, pos1);
            // the next chunk is drawn two stages before this piece's last issue: late enough that a slow SM
            // does not sit on a reserved chunk, early enough that the counter's latency is hidden
            const int draw_at = max(pos, pos1 - 2);
            unsigned long long drawn = 0;
            if (pg.n_chunks > 0 && pos >= pos1 && lane == 0) drawn = atomicAdd(header + kHdrChunk, 1ull);
            // Every piece leaves one record for the finish kernel: the unit it must merge, if any (see below).
            const int piece_pos0 = pos;
            if (pos >= pos1 && lane == 0) piece_info[piece] = make_int4(-1, 0, 0, (int)(unsigned)epoch);
            if (pos < pos1) {  // largest e with prefix[e] <= pos (pieces are drawn in increasing order)
                int lo = e, hi = n_entries;
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (prefix[mid] <= pos) lo = mid; else hi = mid;
                }
                e = lo;
            }
            while (ok && pos < pos1) {
                while (prefix[e + 1] <= pos) ++e;  // skip empty entries
                const int base = prefix[e];
                const int nunits = (prefix[e + 1] - base) / Hkv;
                const int r = pos - base;
                const int c = r / nunits, j = r - c * nunits;
                const int seg_len = min(nunits - j, pos1 - pos);
                const int b = e / S;
                if (e != cur_e) {
                    if (e == nxt_e) clamp_range(nxt_r0, nxt_r1, nxt_len, max_tokens, beg, end);
                    else clamp_range(shard_ranges[2 * e], shard_ranges[2 * e + 1], seq_lens[b], max_tokens, beg, end);
                    cur_e = e;
                    if (e == nxt_tbl_e) { head_tbl = nxt_tbl; head_tbl_e = e; }
                    // start fetching the next non-empty shard's range; it is consumed a segment later
                    int e2 = e + 1;
                    while (e2 < n_entries && prefix[e2 + 1] == prefix[e2]) ++e2;
                    nxt_e = -1;
                    if (e2 < n_entries && prefix[e2] < pos1) {
                        nxt_e = e2;
                        nxt_r0 = shard_ranges[2 * e2];
                        nxt_r1 = shard_ranges[2 * e2 + 1];
                        nxt_len = seq_lens[e2 / S];
                    }
                }
                const int first_page = beg >> 4, last_page = (end - 1) >> 4;
                // the pieces that touch this unit: one segment each, slot = unit + piece (both increase along
                // the unit space, so no two segments share a slot)
                const int p0 = base + c * nunits;
                const int first_piece = piece_of(pg, n_ctas, p0), last_piece = piece_of(pg, n_ctas, p0 + nunits - 1);
                const int nseg = last_piece - first_piece + 1;
                const int first_slot = e * Hkv + c + first_piece;
                if (pos == piece_pos0 && lane == 0)   // does this piece start inside a unit?  (the finish kernel's input)
                    piece_info[piece] = make_int4(j > 0 ? e * Hkv + c : -1, first_slot, nseg, (int)(unsigned)epoch);

                // table entries are fetched 32 pages at a time
                int tbl_page0 = 0, tbl = 0;
                for (int u = 0; ok && u < seg_len; ++u) {
                    const int page0 = first_page + (j + u) * kPagesPerStage;
                    const int np = min(kPagesPerStage, last_page + 1 - page0);
                    if ((u & (32 / kPagesPerStage - 1)) == 0) {
                        tbl_page0 = page0;
                        if (j + u == 0 && head_tbl_e == e) {
                            tbl = head_tbl;           // the shard's first pages: same for every KV head
                        } else {
                            tbl = load_tbl(b, page0, last_page);
                            if (j + u == 0) { head_tbl = tbl; head_tbl_e = e; }
                        }
                    }
                    if (u == 1 && nxt_e >= 0 && nxt_tbl_e != nxt_e) {
                        // the next shard's range has arrived by now: fetch its first table entries too
                        int nb, ne;
                        clamp_range(nxt_r0, nxt_r1, nxt_len, max_tokens, nb, ne);
                        nxt_tbl = load_tbl(nxt_e / S, nb >> 4, (ne - 1) >> 4);
                        nxt_tbl_e = nxt_e;
                    }
                    const int i = lane % kPagesPerStage;    // page within the stage
                    const int part = lane / kPagesPerStage; // 0: K page, 1: V page (>= 2: idle lane)
                    int phys = __shfl_sync(0xffffffffu, tbl, (page0 - tbl_page0) + i);
                    bool bad = false;
                    if (P.check_bounds && (phys < 0 || (long long)phys >= P.num_pages)) { bad = true; phys = 0; }
                    const unsigned bad_mask = __ballot_sync(0xffffffffu, bad && i < np && part == 0) & 0xffu;
                    const bool issuer = (i < np) && (part < 2);

                    if (pg.n_chunks > 0 && pos + u == draw_at && lane == 0) drawn = atomicAdd(header + kHdrChunk, 1ull);
                    if (!mbar_wait(smem_u32(&sm.empty_bar[stage]), phase ^ 1, abort_flag)) { ok = false; break; }
                    const bool first = (u == 0), last = (u == seg_len - 1);
                    const uint32_t full = smem_u32(&sm.full_bar[stage]);
                    if (lane == 0) {
                        StageMeta mt;
                        mt.entry = e; mt.kv_head = c; mt.page0 = page0; mt.npages = np;
                        mt.tok_beg = beg; mt.tok_end = end;
                        mt.flags = (first ? kSegFirst : 0) | (last ? kSegLast : 0) | (nseg << 8);
                        mt.aux = (int)bad_mask;
                        mt.slot = e * Hkv + c + piece;
                        sm.meta[stage] = mt;
                        mbar_arrive_expect_tx(full, (uint32_t)np * 2u * kPageBytes + (first ? (uint32_t)G * 256u : 0u));
                        if (bad_mask) epoch_or(header + kHdrStatus, epoch, kStatusBadPage);
                    }
                    __syncwarp();
                    if (issuer) {
                        const uint32_t dst = smem_u32(&sm.kv[stage][part][i][0]);
                        if (P.kv_nhd)
                            tma_load_page_nhd(dst, part ? &v_map : &k_map, c, phys * kPageSize, full, kv_policy);
                        else
                            tma_load_page(dst, part ? &v_map : &k_map, (phys * Hkv + c) * kPageSize, full, kv_policy);
                    }
                    if (first && lane == 0)
                        bulk_load_1d(smem_u32(&sm.q[stage][0]), q + ((size_t)b * Hq + (size_t)c * G) * kHeadDim,
                                     (uint32_t)G * 256u, full);
                    ++issued;
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
                pos += seg_len;
            }
            if (!ok || pg.n_chunks == 0) break;
            drawn = __shfl_sync(0xffffffffu, drawn, 0);
            if ((drawn >> 20) != (epoch & ((1ull << 44) - 1))) { ok = false; break; }   // not this launch's counter
            const int ticket = (int)(drawn & 0xFFFFFull);
            if (ticket >= pg.n_chunks) break;
            piece = n_ctas + ticket;
        }
        if (ok) {  // end-of-work marker
            // This CTA has issued all of its work: count it now, while the consumer warps finish, so that the
            // arrival's round trips to L2 are off the CTA's exit.  The count only says that every CTA of the
            // launch has started (each read the launch's epoch before its plan), which is all the last arriver
            // needs to know before it bumps the launch count for the NEXT launch.
            if (lane == 0) launch_done(header, epoch, gridDim.x);
            if (mbar_wait(smem_u32(&sm.empty_bar[stage]), phase ^ 1, abort_flag)) {
                if (lane == 0) {
                    StageMeta mt = {};
                    mt.entry = -1;
                    sm.meta[stage] = mt;
                    mbar_arrive(smem_u32(&sm.full_bar[stage]));
                }
            } else ok = false;
        }
        if (!ok) {
            // give up: flag it, then wait (bounded) for the copies still in flight
            if (lane == 0) { sm.abort_flag = 1; epoch_or(header + kHdrStatus, epoch, kStatusTimeout); }
            __syncwarp();
            int s2 = stage;
            uint32_t ph2 = phase;
            for (int k = 0; k < min(issued, kStages); ++k) {
                if (--s2 < 0) { s2 = kStages - 1; ph2 ^= 1; }
                for (unsigned it = 0; it < (1u << 20); ++it)
                    if (mbar_try_wait(smem_u32(&sm.full_bar[s2]), ph2)) break;
            }
        }
        return;
    }

    // ================================ consumer warps ================================
    // empty shards: (0, -inf, -inf), spread over all CTAs' consumer warps while the ring fills
    for (int e = (int)blockIdx.x * kConsumerWarps + warp; e < n_entries; e += (int)gridDim.x * kConsumerWarps) {
        if (prefix[e + 1] != prefix[e]) continue;
        const size_t oe = out_entry(P, e);
        float4 *o4 = reinterpret_cast<float4 *>(o_part + oe * Hq * kHeadDim);
        for (int i = lane; i < Hq * (kHeadDim / 4); i += 32) o4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int h = lane; h < Hq; h += 32) {
            m_part[oe * Hq + h] = neg_inf();
            lse_part[oe * Hq + h] = neg_inf();
        }
    }

    const int g = lane >> 2, t = lane & 3;
    const float scale2 = P.sm_scale * 1.4426950408889634f;  // scores are kept in units of log 2
    const float kLn2 = 0.6931471805599453f;
    uint32_t qf[8][2];
    float m2[2] = {neg_inf(), neg_inf()};
    float l[2] = {0.f, 0.f};
    float acc[8][4];
    int stage = 0;
    uint32_t phase = 0, red_phase0 = 0, red_phase1 = 0;
    const int wp = warp;  // this warp's page within a stage

    // every consumer warp waits on the warp-merge barriers through this; false = abort
    auto red_sync = [&](int which, uint32_t &ph) -> bool {
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sm.red_bar[which]));
        if (!mbar_wait(smem_u32(&sm.red_bar[which]), ph, abort_flag)) {
            if (lane == 0) { sm.abort_flag = 1; epoch_or(header + kHdrStatus, epoch, kStatusTimeout); }
            return false;
        }
        ph ^= 1;
        return true;
    };

    for (;;) {
        if (!mbar_wait(smem_u32(&sm.full_bar[stage]), phase, abort_flag)) {
            if (lane == 0) { sm.abort_flag = 1; epoch_or(header + kHdrStatus, epoch, kStatusTimeout); }
            return;
        }
        const StageMeta mt = sm.meta[stage];
        if (mt.entry < 0) return;   // end of this CTA's work (the producer warp has counted the CTA as done)

        if (mt.flags & kSegFirst) {
            const uint16_t *qs = sm.q[stage];
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                qf[ks][0] = (g < G) ? *reinterpret_cast<const uint32_t *>(qs + g * kHeadDim + ks * 16 + 2 * t) : 0u;
                qf[ks][1] = (g < G) ? *reinterpret_cast<const uint32_t *>(qs + g * kHeadDim + ks * 16 + 2 * t + 8) : 0u;
            }
            m2[0] = m2[1] = neg_inf();
            l[0] = l[1] = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
        }

        if (wp < mt.npages) {
            const int tok0 = (mt.page0 + wp) << 4;
            int tlo = max(mt.tok_beg - tok0, 0), thi = min(mt.tok_end - tok0, kPageSize);
            if ((mt.aux >> wp) & 1) { tlo = 0; thi = 0; }
            const bool ragged = (tlo > 0) || (thi < kPageSize);
            const uint32_t k_base = smem_u32(&sm.kv[stage][0][wp][0]);
            const uint32_t v_base = smem_u32(&sm.kv[stage][1][wp][0]);

            process_page(k_base, v_base, kHalfTileBytes, tlo, thi, ragged, qf, m2, l, acc, scale2, lane);
            if (ragged) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sm.empty_bar[stage]));

        if (mt.flags & kSegLast) {
            // ---- segment epilogue: merge the eight warps' states, four heads per round
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                l[0] += __shfl_xor_sync(0xffffffffu, l[0], off);
                l[1] += __shfl_xor_sync(0xffffffffu, l[1], off);
            }
            constexpr int RG = SweepSmem<G>::kRoundHeads;
            const int nseg = mt.flags >> 8;
            const size_t out_row = out_entry(P, mt.entry) * Hq + (size_t)mt.kv_head * G;  // + head
            float *seg_slot = seg + (size_t)mt.slot * seg_stride;
#pragma unroll
            for (int hr = 0; hr < (G + RG - 1) / RG; ++hr) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int head = 2 * t + hh;
                    if (head < G && head / RG == hr) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            sm.red_acc[warp][head - hr * RG][16 * i + g] = acc[i][hh];
                            sm.red_acc[warp][head - hr * RG][16 * i + g + 8] = acc[i][2 + hh];
                        }
                        if (g == 0) { sm.red_ml[warp][head][0] = m2[hh]; sm.red_ml[warp][head][1] = l[hh]; }
                    }
                }
                if (!red_sync(0, red_phase0)) return;
                // kThreadsPerHead threads share a head: the eight warps' weights are computed once per thread
                // (a group size that is not a multiple of the round leaves the last round's spare threads idle)
                constexpr int kThreadsPerHead = kConsumerThreads / RG;
                const int hl = tid / kThreadsPerHead, d0 = tid % kThreadsPerHead;
                const int head = hr * RG + hl;
                if (hl < RG && head < G) {
                    float M = neg_inf();
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, sm.red_ml[w][head][0]);
                    const bool empty = (M == neg_inf());
                    const float Ms = empty ? 0.f : M;
                    float ew[kConsumerWarps];
                    float z = 0.f;
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) {
                        ew[w] = fast_exp2(sm.red_ml[w][head][0] - Ms);
                        z = fmaf(sm.red_ml[w][head][1], ew[w], z);
                    }
                    const float inv = empty ? 0.f : 1.f / z;
                    for (int d = d0; d < kHeadDim; d += kThreadsPerHead) {
                        float wsum = 0.f;
#pragma unroll
                        for (int w = 0; w < kConsumerWarps; ++w) wsum = fmaf(sm.red_acc[w][hl][d], ew[w], wsum);
                        if (nseg == 1) o_part[(out_row + head) * kHeadDim + d] = wsum * inv;
                        else __stcg(seg_slot + head * kHeadDim + d, wsum);
                    }
                    if (d0 == 0) {
                        if (nseg == 1) {
                            m_part[out_row + head] = empty ? neg_inf() : M * kLn2;
                            lse_part[out_row + head] = empty ? neg_inf() : (M + log2f(z)) * kLn2;
                        } else {
                            __stcg(seg_slot + G * kHeadDim + 2 * head, M);
                            __stcg(seg_slot + G * kHeadDim + 2 * head + 1, z);
                        }
                    }
                }
                if (!red_sync(1, red_phase1)) return;
            }
        }
        if (++stage == kStages) { stage = 0; phase ^= 1; }
    }
}

// ------------------------------------------------------------------ bounded-wait self-test
// Waits, with a short limit, on a barrier that nothing will ever complete, through the same wait
// routine the sweep kernels use: the wait must give up, report QF_STATUS_TIMEOUT and let the kernel
// return, leaving the context usable.
__global__ void selftest_wait_kernel(unsigned long long *header, unsigned long long epoch, unsigned limit)
{
    __shared__ alignas(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        header[kHdrLastEpoch] = epoch;
    }
    __syncthreads();
    if (threadIdx.x == 0 && !mbar_wait(smem_u32(&bar), 0, &abort_flag, limit))
        epoch_or(header + kHdrStatus, epoch, kStatusTimeout);
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// A [2 halves, rows, 64] bf16 view of a KV pool, one 4 KB box per (page, KV head), 128B swizzle.
// box_rows = 16 boxes one (page, KV head) block (4 KB).  For a token-major pool (nhd) the view has a fourth
// dimension, the KV head between the channel half and the token row, and a box takes 16 token rows of one head,
// Hkv rows apart; either way the box lands in shared memory as [half][row][128 B].
inline int make_pool_map(CUtensorMap *out, const void *pool, long long num_pages, int num_kv_heads, int box_rows,
                         bool nhd, char *msg, size_t msg_len)
{
    static EncodeTiledFn encode = nullptr;
    static std::mutex mu;
    struct Entry { const void *pool; long long pages; int heads; int rows; CUtensorMap map; };   // rows < 0: token-major
    // One descriptor per (pointer, shape), hashed by the pointer: a decode loop walks every layer's pools each
    // step, so the cache holds a whole model's worth and a lookup is a handful of probes, not a scan.
    constexpr int kCacheEntries = 1024, kProbes = 8;
    static Entry cache[kCacheEntries];   // zero-initialised: pool == nullptr marks a free entry
    const size_t home = (size_t)(((uintptr_t)pool >> 8) * 0x9E3779B97F4A7C15ull >> 40) % kCacheEntries;
    std::lock_guard<std::mutex> lock(mu);
    const int key_rows = nhd ? -box_rows : box_rows;
    size_t victim = home;
    for (int i = 0; i < kProbes; ++i) {
        Entry &c = cache[(home + i) % kCacheEntries];
        if (c.pool == pool && c.pages == num_pages && c.heads == num_kv_heads && c.rows == key_rows) {
            *out = c.map;
            return 0;
        }
        if (c.pool == nullptr) { victim = (home + i) % kCacheEntries; break; }
    }
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
            snprintf(msg, msg_len, "cuTensorMapEncodeTiled entry point not available");
            return -1;
        }
        encode = (EncodeTiledFn)fn;
    }
    // dims: 64 channels (128 B, the swizzle span), rows (256 B apart), the two halves of a row (128 B apart);
    // a box is one whole 4 KB (page, KV head) block, landing in shared memory as [half][row][128 B]
    const cuuint64_t dims[3] = {64, (cuuint64_t)num_pages * num_kv_heads * kPageSize, 2};
    const cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * 2, 128};
    const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 2};
    // token-major: channels, KV heads (256 B apart), token rows (Hkv x 256 B apart), halves (128 B apart)
    const cuuint64_t dims4[4] = {64, (cuuint64_t)num_kv_heads, (cuuint64_t)num_pages * kPageSize, 2};
    const cuuint64_t strides4[3] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)num_kv_heads * kHeadDim * 2, 128};
    const cuuint32_t box4[4] = {64, 1, (cuuint32_t)box_rows, 2};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUtensorMap map;
    CUresult r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, nhd ? 4 : 3, const_cast<void *>(pool),
                        nhd ? dims4 : dims, nhd ? strides4 : strides, nhd ? box4 : box,
                        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(msg, msg_len, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return -1;
    }
    Entry &slot = cache[victim];   // a free entry among the probes, else the home entry is replaced
    slot.pool = pool; slot.pages = num_pages; slot.heads = num_kv_heads; slot.rows = key_rows; slot.map = map;
    *out = map;
    return 0;
}

// A fresh 54-bit tag per launch: process-random high part, counter low part.
inline unsigned long long next_epoch()
{
    static std::atomic<unsigned long long> counter{
        ((unsigned long long)std::chrono::steady_clock::now().time_since_epoch().count() * 0x9E3779B97F4A7C15ull) >> 10};
    return (counter.fetch_add(1) + 1) & ((1ull << 54) - 1);
}

template <int G>
int launch_sweep_g(const CUtensorMap &kmap, const CUtensorMap &vmap, const void *q, const int32_t *bt,
                   const int32_t *sl, const int32_t *sr, float *o, float *m, float *l, const DevParams &P,
                   char *ws, const WorkspaceLayout &wsl, int n_ctas, unsigned long long epoch, cudaStream_t st,
                   cudaEvent_t ev0, cudaEvent_t ev1, char *msg, size_t msg_len, int *launches, bool skip_finish)
{
    unsigned long long *header = reinterpret_cast<unsigned long long *>(ws + wsl.header_off);
    int *prefix = reinterpret_cast<int *>(ws + wsl.prefix_off);
    int4 *piece_info = reinterpret_cast<int4 *>(ws + wsl.piece_off);
    unsigned long long *counters = reinterpret_cast<unsigned long long *>(ws + wsl.counter_off);
    float *seg = reinterpret_cast<float *>(ws + wsl.seg_off);
    const int n_entries = P.batch * P.max_shards;
    const size_t smem = sizeof(SweepSmem<G>) + 1024;
    {   // per-device kernel attribute, set once under a lock (any host thread may come first)
        static std::mutex attr_mu;
        static bool attr_set[64];
        int dev = 0;
        cudaGetDevice(&dev);
        std::lock_guard<std::mutex> lock(attr_mu);
        if (!attr_set[dev & 63]) {
            cudaError_t e = cudaFuncSetAttribute(sweep_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) { snprintf(msg, msg_len, "cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return -5; }
            attr_set[dev & 63] = true;
        }
    }
    *launches = 0;
    const int *global_prefix = nullptr;
    if (n_entries > kMaxSmemEntries) {
        plan_kernel<<<1, 1024, 0, st>>>(sl, sr, prefix, n_entries, P.max_shards, P.num_kv_heads, P.max_tokens);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) { snprintf(msg, msg_len, "plan_kernel launch: %s", cudaGetErrorString(e)); return -5; }
        global_prefix = prefix;
        *launches += 1;
    }
    if (ev0) cudaEventRecord(ev0, st);
    cudaError_t e = launch_pdl(sweep_kernel<G>, dim3(n_ctas), dim3(kSweepThreads), smem, st, kmap, vmap,
                               (const uint16_t *)q, bt, sl, sr, o, m, l, header, global_prefix, piece_info, seg,
                               wsl.seg_stride, epoch, P);
    if (ev1) cudaEventRecord(ev1, st);
    if (e != cudaSuccess) { snprintf(msg, msg_len, "sweep_kernel launch: %s", cudaGetErrorString(e)); return -5; }
    *launches += 1;
    if (skip_finish) return 0;   // the caller merges the cut units itself (small sweeps: merge_small_kernel)
    // one CTA per piece that can start inside a unit
    e = launch_pdl(finish_kernel<G>, dim3(n_ctas + kMaxDynChunks - 1), dim3(kFinThreads), 0, st,
                   (const int4 *)piece_info, (const unsigned long long *)header, kMaxSweepCtas + kMaxDynChunks,
                   counters, seg, wsl.seg_stride,
                   (int)wsl.seg_slots, o, m, l, n_entries * P.num_kv_heads, P);
    if (e != cudaSuccess) { snprintf(msg, msg_len, "finish_kernel launch: %s", cudaGetErrorString(e)); return -5; }
    *launches += 1;
    return 0;
}

inline int launch_sweep(const void *q, const void *k_cache, const void *v_cache, const int32_t *bt,
                        const int32_t *sl, const int32_t *sr, float *o, float *m, float *l, const DevParams &P,
                        char *ws, const WorkspaceLayout &wsl, int sm_count, unsigned long long epoch,
                        cudaStream_t st, cudaEvent_t ev0, cudaEvent_t ev1, char *msg, size_t msg_len, int *launches,
                        bool skip_finish = false)
{
    CUtensorMap kmap, vmap;
    if (make_pool_map(&kmap, k_cache, P.num_pages, P.num_kv_heads, kPageSize, P.kv_nhd != 0, msg, msg_len)) return -5;
    if (make_pool_map(&vmap, v_cache, P.num_pages, P.num_kv_heads, kPageSize, P.kv_nhd != 0, msg, msg_len)) return -5;
    const int n_ctas = sm_count < kMaxSweepCtas ? sm_count : kMaxSweepCtas;
    switch (P.group) {
    case 1: return launch_sweep_g<1>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, epoch, st, ev0, ev1, msg, msg_len, launches, skip_finish);
    case 2: return launch_sweep_g<2>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, epoch, st, ev0, ev1, msg, msg_len, launches, skip_finish);
    case 3: return launch_sweep_g<3>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, epoch, st, ev0, ev1, msg, msg_len, launches, skip_finish);
    case 4: return launch_sweep_g<4>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, epoch, st, ev0, ev1, msg, msg_len, launches, skip_finish);
    case 5: return launch_sweep_g<5>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, epoch, st, ev0, ev1, msg, msg_len, launches, skip_finish);
    case 6: return launch_sweep_g<6>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, epoch, st, ev0, ev1, msg, msg_len, launches, skip_finish);
    case 7: return launch_sweep_g<7>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, epoch, st, ev0, ev1, msg, msg_len, launches, skip_finish);
    default: return launch_sweep_g<8>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, epoch, st, ev0, ev1, msg, msg_len, launches, skip_finish);
    }
}

}  // namespace qf
