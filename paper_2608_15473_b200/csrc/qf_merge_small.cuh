// The merge of a SMALL sweep in one kernel: the pieces of the (shard, KV head) units that the sweep's schedule
// cut, and then the request's shards (Section 5: states of disjoint sets add, in any order), for a sweep that
// qf_decode_step knows to be small (at most kSmallUnitsPerCta stage units per CTA by a bound the host can compute).
//
// A small sweep is bound by launch and dependent-load latency, not by bandwidth, and what follows it decides its
// latency: the general path runs the finish kernel (piece record, then segments; a second level for units of more
// than eight segments) and then the merge kernel, two kernel boundaries and three to five dependent round trips to
// L2.  Here ONE kernel does both, with one dependent round trip after the sweep (two for long lists):
//
//   before the dependency wait   it redoes the sweep's plan for its request from seq_lens and shard_ranges (inputs
//                                of the step: whatever wrote them finished before the sweep could start), so that
//                                it knows which of its units were cut, into how many segments, and where they lie;
//                                this overlaps the sweep itself
//   after it                     the states it needs are requested in batches that are all in flight together
//                                and merged in a fixed order (bit-deterministic): the cut units' final states
//                                for the caller by one set of CTAs, the request's merged output and log-sum-exp
//                                by another, at the same time, both straight from the sweep's segments.
//
// Merging inside the sweep kernel, by whichever CTA arrives last at a counter, was built and measured first: every
// stage of such a chain costs a fence, an atomic and a CTA barrier (2.5 us each under a profiler) and it lost to
// the three-kernel path by 4-13 us; it was removed.
#pragma once

#include "qf_common.cuh"
#include "qf_finish.cuh"
#include "qf_sweep.cuh"

namespace qf {

#ifndef QF_SMALL_UNITS_PER_CTA
#define QF_SMALL_UNITS_PER_CTA 16
#endif
constexpr int kSmallUnitsPerCta = QF_SMALL_UNITS_PER_CTA;   // a sweep of at most this many stage units per CTA (bound) is "small"
constexpr int kSmallMaxShards  = 32;   // shard slots per request this kernel plans in shared memory

// Can this sweep be treated as small?  Decided on the host from an upper bound on the stage units: every shard of
// every request at the longest length the parameters allow.
inline bool sweep_is_small(const DevParams &P, int n_ctas)
{
    const long long entries = (long long)P.batch * P.max_shards;
    if (entries > kMaxSmemEntries || P.max_shards > kSmallMaxShards) return false;
    const long long pages = ((long long)P.max_tokens + kPageSize - 1) / kPageSize;
    const long long units = entries * P.num_kv_heads * ((pages + kPagesPerStage - 1) / kPagesPerStage);
    return units <= (long long)kSmallUnitsPerCta * n_ctas;
}

// Roles of a CTA, by blockIdx = ((b * Hkv) + c) * (S + 1) + j:
//   j == S   the request role: every state of (request b, KV head c) that the merge counts -- the segments of its
//            cut units and the final states of its uncut shards -- merged in ONE list into out / lse of the group's
//            heads (Section 5: states of disjoint sets add; a cut unit's segments are such states too, so the
//            request's result does not have to wait for the units' own final states);
//   j <  S   the unit role: if the schedule cut unit (b, shard j, c), its segments merged into the unit's final
//            state in the caller's shard arrays; otherwise nothing to do.
// Both roles are the same code: a list of states walked kB at a time, all loads of a batch in flight together,
// merged against the batch's common maximum in list order (the order of every sum is fixed), one destination.
template <int G>
__global__ void __launch_bounds__(kFinThreads)
merge_small_kernel(const int *__restrict__ seq_lens, const int *__restrict__ shard_ranges,
                   const int *__restrict__ shard_counts, const float *__restrict__ seg, int seg_stride, int seg_slots,
                   float *__restrict__ o_part, float *__restrict__ m_part, float *__restrict__ lse_part,
                   float *__restrict__ out, float *__restrict__ lse, int n_sweep_ctas, DevParams P)
{
    constexpr int kB = G <= 2 ? 16 : (G <= 4 ? 8 : 4);   // states whose loads are in flight together
    static_assert(kFinThreads >= kB * 2 * G, "one scalar word per thread and batch");
    __shared__ float s_mz[kB][2 * G];
    __shared__ int s_red[2][kFinThreads / 32];
    __shared__ int s_units[kSmallMaxShards];     // stage units of each shard of this request, all KV heads
    __shared__ int s_first[kSmallMaxShards];     // first segment slot of this KV head's unit of the shard
    __shared__ int s_nseg[kSmallMaxShards];      // segments it was cut into (0: the shard is empty)
    __shared__ int s_items[kSmallMaxShards];     // states of the shard in this CTA's list
    __shared__ const float *s_rows[kB];          // the batch: vector rows (head 0, channel 0), scalars, kind
    __shared__ const float *s_sc[kB];
    __shared__ int s_cut[kB];

    const int d = (int)threadIdx.x, lane = d & 31, warp = d >> 5;
    const int S = P.max_shards, Hkv = P.num_kv_heads, Hq = P.num_q_heads;
    const int bc = (int)blockIdx.x / (S + 1), role = (int)blockIdx.x - bc * (S + 1);
    const int b = bc / Hkv, c = bc - b * Hkv;
    const int n_entries = P.batch * S;
    const float kLn2 = 0.6931471805599453f, kLog2e = 1.4426950408889634f;

    // ---- the plan, from the step's inputs alone (nothing here was written by the sweep)
    int before = 0, all = 0;
    for (int e = d; e < n_entries; e += kFinThreads) {
        const int u = entry_units(seq_lens, shard_ranges, e, S, Hkv, P.max_tokens);
        all += u;
        if (e < b * S) before += u;
        if (e >= b * S && e < (b + 1) * S) s_units[e - b * S] = u;
    }
    for (int off = 16; off > 0; off >>= 1) {
        before += __shfl_xor_sync(0xffffffffu, before, off);
        all += __shfl_xor_sync(0xffffffffu, all, off);
    }
    if (lane == 0) { s_red[0][warp] = before; s_red[1][warp] = all; }
    __syncthreads();
    before = 0; all = 0;
    for (int w = 0; w < kFinThreads / 32; ++w) { before += s_red[0][w]; all += s_red[1][w]; }
    int ns = shard_counts ? shard_counts[b] : S;
    ns = min(max(ns, 0), S);
    if (d < S) {
        const PieceGrid pg = piece_grid(all, n_sweep_ctas, true, P.draw_always != 0);
        int pos = before;
        for (int s = 0; s < d; ++s) pos += s_units[s];
        const int nunits = s_units[d] / Hkv;
        int nseg = 0, first = 0;
        if (nunits > 0) {
            const int p0 = pos + c * nunits;
            const int fp = piece_of(pg, n_sweep_ctas, p0), lp = piece_of(pg, n_sweep_ctas, p0 + nunits - 1);
            nseg = lp - fp + 1;
            first = (b * S + d) * Hkv + c + fp;
            if (nseg > 1 && (first < 0 || (long long)first + nseg > (long long)seg_slots)) nseg = 0;   // cannot happen; never leave the scratch
        }
        s_nseg[d] = nseg;
        s_first[d] = first;
        if (role == S) s_items[d] = (d < ns) ? nseg : 0;               // counted shards: segments, or the one final state
        else s_items[d] = (d == role && nseg > 1) ? nseg : 0;          // the one unit, if it was cut
    }
    __syncthreads();
    int n_items = 0;
    for (int s = 0; s < S; ++s) n_items += s_items[s];
    if (role < S && n_items == 0) return;     // an uncut or empty unit: the sweep wrote its state itself

    grid_dependency_wait();      // from here on: what the sweep wrote
    grid_launch_dependents();

    auto advance = [&](int &s, int &k) {   // the state after (s, k)
        if (++k >= s_items[s]) {
            k = 0;
            do { ++s; } while (s < S && s_items[s] == 0);
        }
    };
    int cs = 0, ck = 0;                      // cursor: shard, state within the shard
    while (cs < S && s_items[cs] == 0) ++cs;
    float acc[G], M[G], z[G];                // running state of the list, channel d of the group's heads (log-2 units)
#pragma unroll
    for (int o = 0; o < G; ++o) { acc[o] = 0.f; M[o] = neg_inf(); z[o] = 0.f; }

    for (int base = 0; base < n_items; base += kB) {
        // the batch's addresses: thread u walks the list to its state (a rolled loop, kept out of the unrolled
        // loads below: this kernel runs once per CTA from cold instruction caches, straight-line length is latency)
        if (d < kB) {
            const float *row = nullptr, *sc = nullptr;
            if (base + d < n_items) {
                int s2 = cs, k2 = ck;
                for (int i = 0; i < d; ++i) advance(s2, k2);
                if (s_nseg[s2] > 1) {
                    row = seg + (size_t)(s_first[s2] + k2) * seg_stride;
                    sc = row + G * kHeadDim;
                } else {
                    const size_t r = out_entry(P, b * S + s2) * Hq + (size_t)c * G;
                    row = o_part + r * kHeadDim;
                    sc = lse_part + r;
                }
            }
            s_rows[d] = row;
            s_sc[d] = sc;
            s_cut[d] = (row != nullptr && sc == row + G * kHeadDim) ? 1 : 0;
        }
        for (int i = 0; i < kB && base + i < n_items; ++i) advance(cs, ck);   // the cursor moves past the batch
        __syncthreads();
        // every load of the batch, back to back
        float av[G][kB];
#pragma unroll
        for (int u = 0; u < kB; ++u) {
            const float *row = s_rows[u];
#pragma unroll
            for (int o = 0; o < G; ++o) av[o][u] = row ? ld_sync_f32(row + o * kHeadDim + d) : 0.f;
        }
        // the batch's scalars, one word per thread: (max, Z) pairs of segments; log Z of a final state as (log2 Z, 1)
        const int u_mine = d / (2 * G), r_mine = d - u_mine * (2 * G);
        float word = (r_mine & 1) ? 0.f : neg_inf();
        if (u_mine < kB && s_rows[u_mine] != nullptr) {
            if (s_cut[u_mine]) word = ld_sync_f32(s_sc[u_mine] + r_mine);
            else word = (r_mine & 1) ? 1.f : ld_sync_f32(s_sc[u_mine] + (r_mine >> 1)) * kLog2e;
        }
        __syncthreads();                       // the previous batch's readers are done with s_mz
        if (u_mine < kB) s_mz[u_mine][r_mine] = word;
        __syncthreads();
#pragma unroll
        for (int o = 0; o < G; ++o) {
            float Mn = M[o];
#pragma unroll
            for (int u = 0; u < kB; ++u) Mn = fmaxf(Mn, s_mz[u][2 * o]);
            const float Ms = (Mn == neg_inf()) ? 0.f : Mn;
            const float keep = fast_exp2(M[o] - Ms);   // 0 while nothing has been merged yet
            z[o] *= keep;
            acc[o] *= keep;
#pragma unroll
            for (int u = 0; u < kB; ++u) {   // fixed order: deterministic
                const float ew = fast_exp2(s_mz[u][2 * o] - Ms);
                z[o] = fmaf(s_mz[u][2 * o + 1], ew, z[o]);
                acc[o] = fmaf(av[o][u], ew, acc[o]);
            }
            M[o] = Mn;
        }
    }

    // ---- the one destination: the request's result, or the unit's final state in the caller's shard arrays
    const size_t unit_row = out_entry(P, b * S + min(role, S - 1)) * Hq + (size_t)c * G;
#pragma unroll
    for (int o = 0; o < G; ++o) {
        const bool empty = (M[o] == neg_inf());
        const float val = empty ? 0.f : acc[o] / z[o];
        const float l = empty ? neg_inf() : (M[o] + log2f(z[o])) * kLn2;
        if (role == S) {
            const size_t bh = (size_t)b * Hq + (size_t)c * G + o;
            out[bh * kHeadDim + d] = val;
            if (d == 0) lse[bh] = l;
        } else {
            o_part[(unit_row + o) * kHeadDim + d] = val;
            if (d == 0) {
                m_part[unit_row + o] = empty ? neg_inf() : M[o] * kLn2;
                lse_part[unit_row + o] = l;
            }
        }
    }
}

// Enqueue the merge of a small sweep: one CTA per (request, KV head).
template <int G>
inline cudaError_t launch_merge_small_g(const int32_t *sl, const int32_t *sr, const int32_t *sc, char *ws,
                                        const WorkspaceLayout &wsl, float *o, float *m, float *l, float *out, float *lse,
                                        int n_sweep_ctas, const DevParams &P, cudaStream_t st)
{
    const float *seg = reinterpret_cast<const float *>(ws + wsl.seg_off);
    // one CTA per (request, KV head, role): S unit roles and the request role
    return launch_pdl(merge_small_kernel<G>, dim3((unsigned)(P.batch * P.num_kv_heads * (P.max_shards + 1))),
                      dim3(kFinThreads), 0, st, sl, sr,
                      sc, seg, wsl.seg_stride, (int)wsl.seg_slots, o, m, l, out, lse, n_sweep_ctas, P);
}
inline cudaError_t launch_merge_small(const int32_t *sl, const int32_t *sr, const int32_t *sc, char *ws,
                                      const WorkspaceLayout &wsl, float *o, float *m, float *l, float *out, float *lse,
                                      int n_sweep_ctas, const DevParams &P, cudaStream_t st)
{
    switch (P.group) {
    case 1: return launch_merge_small_g<1>(sl, sr, sc, ws, wsl, o, m, l, out, lse, n_sweep_ctas, P, st);
    case 2: return launch_merge_small_g<2>(sl, sr, sc, ws, wsl, o, m, l, out, lse, n_sweep_ctas, P, st);
    case 3: return launch_merge_small_g<3>(sl, sr, sc, ws, wsl, o, m, l, out, lse, n_sweep_ctas, P, st);
    case 4: return launch_merge_small_g<4>(sl, sr, sc, ws, wsl, o, m, l, out, lse, n_sweep_ctas, P, st);
    case 5: return launch_merge_small_g<5>(sl, sr, sc, ws, wsl, o, m, l, out, lse, n_sweep_ctas, P, st);
    case 6: return launch_merge_small_g<6>(sl, sr, sc, ws, wsl, o, m, l, out, lse, n_sweep_ctas, P, st);
    case 7: return launch_merge_small_g<7>(sl, sr, sc, ws, wsl, o, m, l, out, lse, n_sweep_ctas, P, st);
    default: return launch_merge_small_g<8>(sl, sr, sc, ws, wsl, o, m, l, out, lse, n_sweep_ctas, P, st);
    }
}

}  // namespace qf

