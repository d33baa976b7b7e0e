// The finish kernel of the cache-side sweep (Section 5: partial states are order-independent): merges the
// (shard, KV head) units that the sweep's piece boundaries cut into segments.
#pragma once

#include "qf_common.cuh"
#include "qf_page_math.cuh"

namespace qf {

// Merges the units that piece boundaries cut into segments, after the sweep (not inside it, by whoever
// arrives last at a counter: a merge is a few round trips to L2, several microseconds each while the
// memory system is saturated, and it would land on the CTAs that are already late).
//
// CTA p looks at the record piece p left.  If the piece starts inside a unit, its segment is the k-th of
// that unit (k >= 1).  Segments are merged in groups of kFinGroup: the CTAs with k == 1 or k a multiple of
// kFinGroup lead a group, the others exit.  A unit of one group is finished by its leader.  Otherwise each
// leader writes its group's partial state over the group's first slot and arrives at the unit's counter;
// the leader that arrives last merges the partials.  Nobody waits for anybody, the depth of a unit of n
// segments is n / kFinGroup^2 batches instead of n / kFinGroup, and the order of every sum is fixed.
// A record is used only if it carries this launch's epoch and its numbers fit the workspace, so an
// aborted sweep cannot make this kernel touch memory outside it.
constexpr int kFinThreads = kHeadDim;   // thread d owns channel d of all G heads
constexpr int kFinGroup   = 8;

// Merge `count` states at slots slot0, slot0 + step, ...: running (acc, M, z) per head for channel d.
// `sync` is the barrier of the threads that take part (it returns false if the wait was abandoned, and the
// merge stops); threads with active == false only keep the barrier count whole.
template <int G, int kB, typename Sync>
__device__ __forceinline__ bool finish_merge_range(const float *__restrict__ seg, int seg_stride, int slot0, int step,
                                                   int count, float (*s_mz)[2 * G], float *acc, float *M, float *z, int d,
                                                   bool active, Sync &&sync)
{
    // kB: states whose loads are in flight together
#pragma unroll
    for (int o = 0; o < G; ++o) { acc[o] = 0.f; M[o] = neg_inf(); z[o] = 0.f; }
    for (int base = 0; base < count; base += kB) {
        float av[G][kB];
        float mz = 0.f;
        const int u_mine = d / (2 * G), r_mine = d % (2 * G);   // (M, z) pairs of the batch: one word per thread
        const bool mz_on = active && u_mine < kB && base + u_mine < count;
        if (active) {
#pragma unroll
            for (int u = 0; u < kB; ++u) {
                const bool on = base + u < count;
                const float *sl = seg + (size_t)(slot0 + (on ? base + u : 0) * step) * seg_stride;
#pragma unroll
                for (int o = 0; o < G; ++o) av[o][u] = on ? ld_sync_f32(sl + o * kHeadDim + d) : 0.f;
            }
            if (mz_on) mz = ld_sync_f32(seg + (size_t)(slot0 + (base + u_mine) * step) * seg_stride + G * kHeadDim + r_mine);
        }
        if (!sync()) return false;             // the previous batch's readers are done with s_mz
        if (active && u_mine < kB) s_mz[u_mine][r_mine] = mz_on ? mz : (r_mine & 1 ? 0.f : neg_inf());
        if (!sync()) return false;
        if (active) {
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
    }
    return true;
}

template <int G>
__global__ void __launch_bounds__(kFinThreads)
finish_kernel(const int4 *__restrict__ piece_info, const unsigned long long *__restrict__ header,
              int max_pieces, unsigned long long *__restrict__ counters, float *__restrict__ seg, int seg_stride,
              int seg_slots,
              float *__restrict__ o_part, float *__restrict__ m_part, float *__restrict__ lse_part, int n_units,
              DevParams P)
{
    constexpr int kFinBatch = (G == 8) ? 4 : 8;
    static_assert(kFinThreads >= 8 * 2 * G, "one (M, z) word per thread and batch");
    __shared__ float s_mz[8][2 * G];
    __shared__ int s_last;
    grid_dependency_wait();
    grid_launch_dependents();
    const int d = (int)threadIdx.x;
    const int p = (int)blockIdx.x + 1;      // piece 0 cannot start inside a unit
    const int n_pieces = (int)(ld_sync_u64(header + kHdrTotals) >> 32);
    const int4 rec = ld_sync_int4(piece_info + min(p, max_pieces - 1));
    const unsigned long long epoch = ld_sync_u64(header + kHdrLastEpoch);
    if (p >= n_pieces || rec.x < 0 || rec.w != (int)(unsigned)epoch) return;
    const int unit = rec.x, first_slot = rec.y, nseg = rec.z;
    if (unit >= n_units || nseg < 2 || first_slot < 0 || (long long)first_slot + nseg > (long long)seg_slots) return;
    const int k = unit + p - first_slot;    // this piece's segment is the k-th of the unit
    if (k < 1 || k >= nseg) return;
    if (k != 1 && (k % kFinGroup) != 0) return;
    const int group = k / kFinGroup, n_groups = (nseg + kFinGroup - 1) / kFinGroup;
    const int seg0 = group * kFinGroup;
    const int Hkv = P.num_kv_heads, Hq = P.num_q_heads;
    const size_t out_row = out_entry(P, unit / Hkv) * Hq + (size_t)(unit % Hkv) * G;
    const float kLn2 = 0.6931471805599453f;

    float acc[G], M[G], z[G];
    auto write_final = [&]() {
#pragma unroll
        for (int o = 0; o < G; ++o) {
            const bool empty = (M[o] == neg_inf());
            o_part[(out_row + o) * kHeadDim + d] = empty ? 0.f : acc[o] / z[o];
            if (d == 0) {
                m_part[out_row + o] = empty ? neg_inf() : M[o] * kLn2;
                lse_part[out_row + o] = empty ? neg_inf() : (M[o] + log2f(z[o])) * kLn2;
            }
        }
    };
    auto cta_sync = []() -> bool { __syncthreads(); return true; };
    finish_merge_range<G, kFinBatch>(seg, seg_stride, first_slot + seg0, 1, min(kFinGroup, nseg - seg0), s_mz, acc, M, z, d, true, cta_sync);
    if (n_groups == 1) { write_final(); return; }

    // the group's partial state replaces the group's first segment (which only this CTA reads)
    float *slot = seg + (size_t)(first_slot + seg0) * seg_stride;
#pragma unroll
    for (int o = 0; o < G; ++o) {
        __stcg(slot + o * kHeadDim + d, acc[o]);
        if (d == 0) { __stcg(slot + G * kHeadDim + 2 * o, M[o]); __stcg(slot + G * kHeadDim + 2 * o + 1, z[o]); }
    }
    __syncthreads();
    if (d == 0) {
        __threadfence();
        s_last = (epoch_arrive(counters + unit, epoch) == (unsigned)n_groups) ? 1 : 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    finish_merge_range<G, kFinBatch>(seg, seg_stride, first_slot, kFinGroup, n_groups, s_mz, acc, M, z, d, true, cta_sync);
    write_final();
}

}  // namespace qf
