// Head-parallel sweep: the persistent streaming kernel for caches whose KV-head count is a
// multiple of eight (the Qwen3 shapes).
//
// Same plan / stream / merge structure as sweep_kernel (qf_sweep.cuh), but a ring stage holds ONE
// page of EIGHT KV heads, and consumer warp w owns KV head w of the stage's head group for the whole
// sweep.  Consequences:
//   - a stage is two 32 KB TMA boxes (K and V of the page: 8 heads x 16 rows x 256 B are contiguous
//     in the pool), one block-table entry per stage;
//   - a warp's online-softmax state covers a whole (shard, KV head) segment by itself, so a segment
//     ends with a warp-local epilogue: no cross-warp merge, no CTA barrier anywhere in the sweep;
//   - the unit space (pages x head groups, in request order) is cut into one equal piece per CTA.
//     A (shard, KV head) unit cut by a piece boundary is merged by the warp that arrives last at the
//     unit's epoch-tagged counter.  A piece owns two groups of eight segment slots: group 2p for the
//     unit that started in an earlier piece, group 2p+1 for the unit that starts in piece p and runs
//     past its end; at most one unit of each kind exists per piece.
//   Measured on B200: with the ring always full the memory system does not share bandwidth equally
//   between SMs, which costs this kernel a ~10 % tail on long shards; it wins when shards are short
//   (many segment ends), which is why it is opt-in (QF_FLAG_HEAD_PARALLEL).
#pragma once

#include "qf_sweep.cuh"

namespace qf {

constexpr int kHpHeads = 8;                              // KV heads per stage, one per consumer warp
constexpr int kHpTileBytes = kHpHeads * kPageBytes;      // 32 KB: K (or V) of one page, eight heads
constexpr int kHpHalfStride = kHpTileBytes / 2;          // the two 64-channel halves of the box
constexpr int kHpStages = 3;

template <int G>
struct HpSmem {
    alignas(1024) uint8_t kv[kHpStages][2][kHpTileBytes];  // [stage][K|V][half][head][row][128B], swizzled
    alignas(16) uint16_t q[kHpStages][kHpHeads * G * kHeadDim];
    alignas(16) StageMeta meta[kHpStages];
    alignas(8) unsigned long long full_bar[kHpStages];
    alignas(8) unsigned long long empty_bar[kHpStages];
    int abort_flag;
    unsigned long long epoch;   // this launch's epoch, read once per CTA
    int scan_ws[kConsumerWarps + 1];
    int prefix[kMaxSmemEntries + 1];
};

// Geometry of the pieces the unit space [0, total) is cut into: one equal piece per CTA.
struct Pieces {
    int total, qs;
    __device__ __forceinline__ void init(int total_, int n_ctas)
    {
        total = total_;
        qs = max(1, (total + n_ctas - 1) / n_ctas);
    }
    __device__ __forceinline__ int piece_of(int pos) const { return pos / qs; }
    __device__ __forceinline__ int start(int p) const { return min(p * qs, total); }
    __device__ __forceinline__ int end(int p) const { return min((p + 1) * qs, total); }
};

// Merge the segments a (shard, KV head) unit was cut into, pieces p_first .. p_first+nseg-1, in that
// order (deterministic), by the one warp that arrived last.
template <int G>
__device__ __forceinline__ void merge_pieces(const float *__restrict__ seg, int seg_stride, int p_first, int nseg,
                                             int head_in_group, size_t out_row, float *__restrict__ o_part,
                                             float *__restrict__ m_part, float *__restrict__ lse_part, int lane)
{
    const float kLn2 = 0.6931471805599453f;
    auto slot_of = [&](int i) -> const float * {
        return seg + (size_t)((2 * (p_first + i) + (i == 0 ? 1 : 0)) * kHpHeads + head_in_group) * seg_stride;
    };
    constexpr int kBatch = 8;   // segments whose loads are in flight together
    for (int idx = lane; idx < G * kHeadDim; idx += 32) {
        const int head = idx >> 7, d = idx & 127;
        float M = neg_inf();
        for (int base = 0; base < nseg; base += kBatch) {
            float mv[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u)
                mv[u] = (base + u < nseg) ? ld_sync_f32(slot_of(base + u) + G * kHeadDim + 2 * head) : neg_inf();
#pragma unroll
            for (int u = 0; u < kBatch; ++u) M = fmaxf(M, mv[u]);
        }
        const bool empty = (M == neg_inf());
        const float Ms = empty ? 0.f : M;
        float z = 0.f, wsum = 0.f;
        for (int base = 0; base < nseg; base += kBatch) {
            float mv[kBatch], zv[kBatch], av[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const bool on = base + u < nseg;
                const float *sl = slot_of(on ? base + u : 0);
                mv[u] = on ? ld_sync_f32(sl + G * kHeadDim + 2 * head) : neg_inf();
                zv[u] = on ? ld_sync_f32(sl + G * kHeadDim + 2 * head + 1) : 0.f;
                av[u] = on ? ld_sync_f32(sl + head * kHeadDim + d) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {   // fixed order: deterministic
                const float ew = fast_exp2(mv[u] - Ms);
                z = fmaf(zv[u], ew, z);
                wsum = fmaf(av[u], ew, wsum);
            }
        }
        o_part[(out_row + head) * kHeadDim + d] = empty ? 0.f : wsum / z;
        if (d == 0) {
            m_part[out_row + head] = empty ? neg_inf() : M * kLn2;
            lse_part[out_row + head] = empty ? neg_inf() : (M + log2f(z)) * kLn2;
        }
    }
}

template <int G>
__global__ void __launch_bounds__(kSweepThreads, 1)
sweep_hp_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
                const uint16_t *__restrict__ q, const int *__restrict__ block_table,
                const int *__restrict__ seq_lens, const int *__restrict__ shard_ranges,
                float *__restrict__ o_part, float *__restrict__ m_part, float *__restrict__ lse_part,
                unsigned long long *__restrict__ header, const int *__restrict__ global_prefix,
                unsigned long long *__restrict__ counters, float *__restrict__ seg, int seg_stride,
                unsigned long long host_epoch, DevParams P)
{
    extern __shared__ uint8_t smem_raw[];
    HpSmem<G> &sm = *reinterpret_cast<HpSmem<G> *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int S = P.max_shards, Hkv = P.num_kv_heads, Hq = P.num_q_heads;
    const int n_groups = Hkv / kHpHeads;
    const int n_entries = P.batch * S;
    volatile int *abort_flag = &sm.abort_flag;

    if (tid == 0) {
        for (int s = 0; s < kHpStages; ++s) {
            mbar_init(smem_u32(&sm.full_bar[s]), 1);
            mbar_init(smem_u32(&sm.empty_bar[s]), kConsumerWarps);
        }
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    grid_dependency_wait();     // nothing above touches global memory
    grid_launch_dependents();
    if (tid == 0) {
        sm.epoch = launch_epoch(header, host_epoch);
        if (blockIdx.x == 0) header[kHdrLastEpoch] = sm.epoch;
    }

    // ---- plan: prefix sum of pages x head groups over (request, shard) entries
    const int *prefix;
    if (global_prefix) {
        prefix = global_prefix;
        __syncthreads();
    } else {
        int carry = 0;
        for (int base = 0; base < n_entries; base += kConsumerThreads) {
            const int e = base + tid;
            const int cnt = (tid < kConsumerThreads && e < n_entries)
                                ? entry_units(seq_lens, shard_ranges, e, S, Hkv, n_groups) : 0;
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
    const int total = prefix[n_entries];
    Pieces pc;
    pc.init(total, (int)gridDim.x);
    if (blockIdx.x == 0 && tid == 0)
        header[kHdrTotals] = (unsigned long long)(unsigned)total | ((unsigned long long)(unsigned)pc.qs << 32);

    if (warp == kConsumerWarps) {
        // ============================ producer warp ============================
        const unsigned long long kv_policy = l2_evict_first_policy();
        int stage = 0;
        uint32_t phase = 0;
        int issued = 0;
        bool ok = true;
        const int piece = (int)blockIdx.x;
        const int pos1 = pc.end(piece);
        int pos = pc.start(piece);
        int e = 0;
        {  // largest e with prefix[e] <= pos
            int lo = 0, hi = n_entries;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (prefix[mid] <= pos) lo = mid; else hi = mid;
            }
            e = lo;
        }
        while (ok && pos < pos1) {
            while (prefix[e + 1] <= pos) ++e;  // skip empty entries
            const int base = prefix[e];
            const int npages = (prefix[e + 1] - base) / n_groups;
            const int r = pos - base;
            const int grp = r / npages, j = r - grp * npages;
            const int seg_len = min(npages - j, pos1 - pos);
            const int b = e / S;
            int beg, end;
            clamp_range(shard_ranges[2 * e], shard_ranges[2 * e + 1], seq_lens[b], beg, end);
            const int first_page = beg >> 4, last_page = (end - 1) >> 4;
            // the pieces that touch this (shard, head group): one segment each
            const int u0 = base + grp * npages;
            const int p_first = pc.piece_of(u0);
            const int nseg = pc.piece_of(u0 + npages - 1) - p_first + 1;
            const long long row_base = (long long)b * P.max_pages_per_req;

            int tbl_page0 = 0, tbl = 0;  // table entries are fetched 32 pages at a time
            for (int u = 0; ok && u < seg_len; ++u) {
                const int page = first_page + j + u;
                if ((u & 31) == 0) {
                    tbl_page0 = page;
                    const int lp = min(page + lane, last_page);
                    tbl = block_table ? block_table[row_base + lp] : (int)(row_base + lp);
                }
                int phys = __shfl_sync(0xffffffffu, tbl, page - tbl_page0);
                bool bad = false;
                if (P.check_bounds && (phys < 0 || (long long)phys >= P.num_pages)) { bad = true; phys = 0; }

                if (!mbar_wait(smem_u32(&sm.empty_bar[stage]), phase ^ 1, abort_flag)) { ok = false; break; }
                const bool first = (u == 0), last = (u == seg_len - 1);
                const uint32_t full = smem_u32(&sm.full_bar[stage]);
                if (lane == 0) {
                    StageMeta mt;
                    mt.entry = e; mt.kv_head = grp * kHpHeads; mt.page0 = page; mt.npages = piece;
                    mt.tok_beg = beg; mt.tok_end = end;
                    mt.flags = (first ? kSegFirst : 0) | (last ? kSegLast : 0) | (nseg << 8);
                    mt.aux = (bad ? 1 : 0) | (p_first << 8);
                    sm.meta[stage] = mt;
                    mbar_arrive_expect_tx(full, 2u * kHpTileBytes + (first ? (uint32_t)(kHpHeads * G) * 256u : 0u));
                    if (bad) epoch_or(header + kHdrStatus, epoch, kStatusBadPage);
                }
                __syncwarp();
                if (lane < 2) {    // two 32 KB boxes: K and V of the page, eight heads each
                    const int row = (phys * Hkv + grp * kHpHeads) * kPageSize;
                    tma_load_page(smem_u32(&sm.kv[stage][lane][0]), lane ? &v_map : &k_map, row, full, kv_policy);
                } else if (lane == 2 && first) {
                    bulk_load_1d(smem_u32(&sm.q[stage][0]),
                                 q + ((size_t)b * Hq + (size_t)grp * kHpHeads * G) * kHeadDim,
                                 (uint32_t)(kHpHeads * G) * 256u, full);
                }
                ++issued;
                if (++stage == kHpStages) { stage = 0; phase ^= 1; }
            }
            pos += seg_len;
        }
        if (ok) {  // end-of-work marker
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
            for (int k = 0; k < min(issued, kHpStages); ++k) {
                if (--s2 < 0) { s2 = kHpStages - 1; ph2 ^= 1; }
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
        float4 *o4 = reinterpret_cast<float4 *>(o_part + (size_t)e * Hq * kHeadDim);
        for (int i = lane; i < Hq * (kHeadDim / 4); i += 32) o4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int h = lane; h < Hq; h += 32) {
            m_part[(size_t)e * Hq + h] = neg_inf();
            lse_part[(size_t)e * Hq + h] = neg_inf();
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
    uint32_t phase = 0;

    for (;;) {
        if (!mbar_wait(smem_u32(&sm.full_bar[stage]), phase, abort_flag)) {
            if (lane == 0) { sm.abort_flag = 1; epoch_or(header + kHdrStatus, epoch, kStatusTimeout); }
            return;
        }
        const StageMeta mt = sm.meta[stage];
        if (mt.entry < 0) {   // end of this CTA's piece
            if (tid == 0) launch_done(header, epoch, gridDim.x);
            return;
        }

        if (mt.flags & kSegFirst) {
            const uint16_t *qs = sm.q[stage] + warp * G * kHeadDim;  // this warp's head group rows
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

        {
            const int tok0 = mt.page0 << 4;
            int tlo = max(mt.tok_beg - tok0, 0), thi = min(mt.tok_end - tok0, kPageSize);
            if (mt.aux & 1) { tlo = 0; thi = 0; }
            const bool ragged = (tlo > 0) || (thi < kPageSize);
            const uint32_t k_base = smem_u32(&sm.kv[stage][0][warp * kHalfTileBytes]);
            const uint32_t v_base = smem_u32(&sm.kv[stage][1][warp * kHalfTileBytes]);
            process_page(k_base, v_base, kHpHalfStride, tlo, thi, ragged, qf, m2, l, acc, scale2, lane);
            if (ragged) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sm.empty_bar[stage]));

        if (mt.flags & kSegLast) {
            // ---- warp-local epilogue: this warp alone holds the state of (shard, KV head) for its segment
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                l[0] += __shfl_xor_sync(0xffffffffu, l[0], off);
                l[1] += __shfl_xor_sync(0xffffffffu, l[1], off);
            }
            const int nseg = mt.flags >> 8;
            const int c = mt.kv_head + warp;
            const int unit = mt.entry * Hkv + c;
            const size_t out_row = (size_t)mt.entry * Hq + (size_t)c * G;  // + head
            if (nseg == 1) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int head = 2 * t + hh;
                    if (head < G) {
                        const bool empty = (m2[hh] == neg_inf());
                        const float inv = empty ? 0.f : 1.f / l[hh];
                        float *o = o_part + (out_row + head) * kHeadDim;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            o[16 * i + g] = acc[i][hh] * inv;
                            o[16 * i + g + 8] = acc[i][2 + hh] * inv;
                        }
                        if (g == 0) {
                            m_part[out_row + head] = empty ? neg_inf() : m2[hh] * kLn2;
                            lse_part[out_row + head] = empty ? neg_inf() : (m2[hh] + log2f(l[hh])) * kLn2;
                        }
                    }
                }
            } else {
                // the unit was cut by slice boundaries: park this segment's state, and merge all of the
                // unit's segments if this warp is the last to arrive
                const int my_piece = mt.npages, p_first = mt.aux >> 8;
                float *slot = seg + (size_t)((2 * my_piece + (my_piece == p_first ? 1 : 0)) * kHpHeads + warp) * seg_stride;
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int head = 2 * t + hh;
                    if (head < G) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            __stcg(slot + head * kHeadDim + 16 * i + g, acc[i][hh]);
                            __stcg(slot + head * kHeadDim + 16 * i + g + 8, acc[i][2 + hh]);
                        }
                        if (g == 0) {
                            __stcg(slot + G * kHeadDim + 2 * head, m2[hh]);
                            __stcg(slot + G * kHeadDim + 2 * head + 1, l[hh]);
                        }
                    }
                }
                __threadfence();
                __syncwarp();
                unsigned n = 0;
                if (lane == 0) {
                    n = epoch_arrive(counters + unit, epoch);
                    if (n == 0) epoch_or(header + kHdrStatus, epoch, kStatusTimeout);
                }
                n = __shfl_sync(0xffffffffu, n, 0);
                if (n == (unsigned)nseg) {
                    __threadfence();
                    merge_pieces<G>(seg, seg_stride, p_first, nseg, warp, out_row, o_part, m_part, lse_part, lane);
                }
            }
        }
        if (++stage == kHpStages) { stage = 0; phase ^= 1; }
    }
}

template <int G>
int launch_sweep_hp_g(const CUtensorMap &kmap, const CUtensorMap &vmap, const void *q, const int32_t *bt,
                      const int32_t *sl, const int32_t *sr, float *o, float *m, float *l, const DevParams &P,
                      char *ws, const WorkspaceLayout &wsl, int n_ctas, unsigned long long epoch,
                      cudaStream_t st, cudaEvent_t ev0, cudaEvent_t ev1, char *msg, size_t msg_len, int *launches)
{
    unsigned long long *header = reinterpret_cast<unsigned long long *>(ws + wsl.header_off);
    int *prefix = reinterpret_cast<int *>(ws + wsl.prefix_off);
    unsigned long long *counters = reinterpret_cast<unsigned long long *>(ws + wsl.counter_off);
    float *seg = reinterpret_cast<float *>(ws + wsl.seg_off);
    const int n_entries = P.batch * P.max_shards;
    const size_t smem = sizeof(HpSmem<G>) + 1024;
    static bool attr_set[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set[dev & 63]) {
        cudaError_t e = cudaFuncSetAttribute(sweep_hp_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) { snprintf(msg, msg_len, "cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return -5; }
        attr_set[dev & 63] = true;
    }
    *launches = 0;
    const int *global_prefix = nullptr;
    if (n_entries > kMaxSmemEntries) {
        plan_kernel<<<1, 1024, 0, st>>>(sl, sr, prefix, n_entries, P.max_shards, P.num_kv_heads,
                                        P.num_kv_heads / kHpHeads);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) { snprintf(msg, msg_len, "plan_kernel launch: %s", cudaGetErrorString(e)); return -5; }
        global_prefix = prefix;
        *launches += 1;
    }
    if (ev0) cudaEventRecord(ev0, st);
    cudaError_t e = launch_pdl(sweep_hp_kernel<G>, dim3(n_ctas), dim3(kSweepThreads), smem, st, kmap, vmap,
                               (const uint16_t *)q, bt, sl, sr, o, m, l, header, global_prefix, counters, seg,
                               wsl.seg_stride, epoch, P);
    if (ev1) cudaEventRecord(ev1, st);
    if (e != cudaSuccess) { snprintf(msg, msg_len, "sweep_hp_kernel launch: %s", cudaGetErrorString(e)); return -5; }
    *launches += 1;
    return 0;
}

// Picks the kernel: the unit kernel, or the head-parallel kernel when asked for and applicable.
inline int launch_sweep_any(const void *q, const void *k_cache, const void *v_cache, const int32_t *bt,
                            const int32_t *sl, const int32_t *sr, float *o, float *m, float *l, const DevParams &P,
                            char *ws, const WorkspaceLayout &wsl, int sm_count, unsigned long long epoch,
                            bool want_hp, cudaStream_t st, cudaEvent_t ev0, cudaEvent_t ev1,
                            char *msg, size_t msg_len, int *launches)
{
    const bool hp = want_hp && (P.num_kv_heads % kHpHeads == 0) && P.group <= 4;
    if (!hp)
        return launch_sweep(q, k_cache, v_cache, bt, sl, sr, o, m, l, P, ws, wsl, sm_count, epoch, st, ev0, ev1, msg,
                            msg_len, launches);
    CUtensorMap kmap, vmap;
    const int box_rows = kHpHeads * kPageSize;
    if (make_pool_map(&kmap, k_cache, P.num_pages, P.num_kv_heads, box_rows, msg, msg_len)) return -5;
    if (make_pool_map(&vmap, v_cache, P.num_pages, P.num_kv_heads, box_rows, msg, msg_len)) return -5;
    const int n_ctas = sm_count < kMaxSweepCtas ? sm_count : kMaxSweepCtas;
    switch (P.group) {
    case 1: return launch_sweep_hp_g<1>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, epoch, st, ev0, ev1, msg, msg_len, launches);
    case 2: return launch_sweep_hp_g<2>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, epoch, st, ev0, ev1, msg, msg_len, launches);
    default: return launch_sweep_hp_g<4>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, epoch, st, ev0, ev1, msg, msg_len, launches);
    }
}

}  // namespace qf
