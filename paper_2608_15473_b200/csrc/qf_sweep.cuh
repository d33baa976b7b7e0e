// The staged sweep: plan -> persistent TMA/tensor-core sweep -> segment merge.
//
// Section 5 of the Q-First paper lets a cache be split anywhere: partial states
// (W, Z) add over disjoint token sets.  The user-visible split is the shard; this
// file splits further, invisibly, so that every SM streams the same number of KV
// bytes whatever the batch looks like:
//
//   plan_kernel   turns (seq_lens, shard_ranges) into a prefix sum over
//                 "stage units" (8 pages = 128 tokens of one KV head of one shard);
//   sweep_kernel  one persistent CTA per SM takes an equal contiguous slice of the
//                 unit space.  A producer warp walks the slice, looks pages up in
//                 the block table and issues TMA tile loads (128B-swizzled) into a
//                 3-stage shared-memory ring; 8 consumer warps each take one page of
//                 a stage: S = K Q^T on tensor cores (tokens on M, the group's heads
//                 on N), fp32 online softmax, P split into bf16 hi+lo, O^T += V^T P^T.
//                 A slice boundary inside a shard yields a segment state in scratch;
//   merge_kernel  merges the segments of a (shard, KV head) into o_part/m_part/
//                 lse_part, and writes the empty-shard convention.
//
// All waits are bounded: a wait that runs out sets QF_STATUS_TIMEOUT, raises a
// CTA-wide abort flag and every warp leaves through the same exit.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>

#include "qf_common.cuh"

namespace qf {

constexpr int kPagesPerStage = 8;                 // one page per consumer warp
constexpr int kConsumerWarps = kPagesPerStage;
constexpr int kSweepThreads  = (kConsumerWarps + 1) * 32;
constexpr int kStages        = 3;
constexpr int kMaxSweepCtas  = 512;               // bound used for scratch sizing
constexpr int kHalfTileBytes = 2048;              // 16 rows x 64 channels of bf16
constexpr int kStageKVBytes  = kPagesPerStage * kPageBytes * 2;  // K and V
constexpr int kRedStride     = kHeadDim + 4;      // padded row of the warp-merge buffer
constexpr unsigned kSpinLimit = 1u << 24;

struct WorkspaceLayout {
    size_t header_off, prefix_off, seg_off, total;
    int seg_stride;  // floats per segment slot
};

// Header words (int32) at the start of the workspace.
enum { kHdrStatus = 0, kHdrTotalUnits = 1, kHdrUnitsPerCta = 2 };

inline int seg_stride_floats(int G) { return G * kHeadDim + ((2 * G + 3) & ~3); }

inline WorkspaceLayout workspace_layout(int batch, int max_shards, int num_kv_heads, int G)
{
    WorkspaceLayout L;
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t entries = (size_t)batch * max_shards;
    L.header_off = 0;
    L.prefix_off = 256;
    L.seg_off = up(L.prefix_off + (entries + 1) * sizeof(int));
    L.seg_stride = seg_stride_floats(G);
    const size_t slots = entries * num_kv_heads + kMaxSweepCtas;
    L.total = up(L.seg_off + slots * L.seg_stride * sizeof(float));
    return L;
}

// ------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if the limit ran out or another warp aborted.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    for (unsigned it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 64) {
            if (*abort_flag) return false;
            __nanosleep(64);
        }
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
// D = A(16x16, row) * B(16x8, col) + D, bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// ------------------------------------------------------------------ plan kernel
// prefix[e] = number of stage units (x Hkv) before entry e = b*S + s.
__global__ void __launch_bounds__(1024)
plan_kernel(const int *__restrict__ seq_lens, const int *__restrict__ shard_ranges, int *__restrict__ header,
            int *__restrict__ prefix, int n_entries, int max_shards, int num_kv_heads, int n_ctas)
{
    __shared__ int warp_sums[32];
    __shared__ int carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (int base = 0; base < n_entries; base += 1024) {
        const int e = base + tid;
        int cnt = 0;
        if (e < n_entries) {
            int beg, end;
            clamp_range(shard_ranges[2 * e], shard_ranges[2 * e + 1], seq_lens[e / max_shards], beg, end);
            if (end > beg) {
                const int npages = ((end - 1) >> 4) - (beg >> 4) + 1;
                cnt = ((npages + kPagesPerStage - 1) / kPagesPerStage) * num_kv_heads;
            }
        }
        int x = cnt;  // inclusive scan within the warp
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, x, off);
            if (lane >= off) x += y;
        }
        if (lane == 31) warp_sums[warp] = x;
        __syncthreads();
        if (warp == 0) {
            int w = warp_sums[lane];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, w, off);
                if (lane >= off) w += y;
            }
            warp_sums[lane] = w;  // inclusive over warps
        }
        __syncthreads();
        const int carry = carry_s;
        const int excl = carry + (warp ? warp_sums[warp - 1] : 0) + x - cnt;
        if (e < n_entries) prefix[e] = excl;
        __syncthreads();
        if (tid == 1023) carry_s = carry + warp_sums[31];
        __syncthreads();
    }
    if (tid == 0) {
        const int total = carry_s;
        prefix[n_entries] = total;
        header[kHdrStatus] = 0;
        header[kHdrTotalUnits] = total;
        header[kHdrUnitsPerCta] = (total + n_ctas - 1) / n_ctas;
    }
}

// ------------------------------------------------------------------ sweep kernel
struct __align__(16) StageMeta {
    int entry;     // b*S + s; -1 = no more work
    int kv_head;
    int page0;     // first logical page of this stage
    int npages;    // 1..8
    int tok_beg;   // clamped shard range
    int tok_end;
    int flags;     // bit0 first stage of a segment, bit1 last stage, bit2 segment == whole unit
    int aux;       // bits 0..7: pages whose table entry was out of range; bits 8..: segment slot
};
enum { kSegFirst = 1, kSegLast = 2, kSegWhole = 4 };

template <int G>
struct SweepSmem {
    // every K/V half tile is a 1024-byte-aligned 128B-swizzled TMA destination
    alignas(1024) uint8_t kv[kStages][2][kPagesPerStage][kPageBytes];  // [stage][K|V][page][half][row][128B]
    alignas(16) uint16_t q[kStages][8 * kHeadDim];
    static constexpr int kRoundHeads = G < 4 ? G : 4;  // heads merged per epilogue round
    alignas(16) float red_acc[kConsumerWarps][kRoundHeads][kRedStride];
    alignas(16) float red_ml[kConsumerWarps][G][2];
    alignas(16) StageMeta meta[kStages];
    alignas(8) unsigned long long full_bar[kStages];
    alignas(8) unsigned long long empty_bar[kStages];
    alignas(8) unsigned long long red_bar[2];
    int abort_flag;
};

template <int G>
__global__ void __launch_bounds__(kSweepThreads, 1)
sweep_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
             const uint16_t *__restrict__ q, const int *__restrict__ block_table,
             const int *__restrict__ seq_lens, const int *__restrict__ shard_ranges,
             float *__restrict__ o_part, float *__restrict__ m_part, float *__restrict__ lse_part,
             int *__restrict__ header, const int *__restrict__ prefix, float *__restrict__ seg,
             int seg_stride, DevParams P)
{
    extern __shared__ uint8_t smem_raw[];
    SweepSmem<G> &sm = *reinterpret_cast<SweepSmem<G> *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int S = P.max_shards, Hkv = P.num_kv_heads, Hq = P.num_q_heads;
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
    __syncthreads();

    const int total = header[kHdrTotalUnits];
    const int per_cta = header[kHdrUnitsPerCta];
    const long long pos0_ll = (long long)blockIdx.x * per_cta;
    const int pos0 = (int)min((long long)total, pos0_ll);
    const int pos1 = (int)min((long long)total, pos0_ll + per_cta);

    if (warp == kConsumerWarps) {
        // ============================ producer warp ============================
        int stage = 0;
        uint32_t phase = 0;
        int issued = 0;
        bool ok = true;
        const int n_entries = P.batch * S;
        int pos = pos0;
        int e = 0;
        if (pos < pos1) {  // largest e with prefix[e] <= pos
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
            const int nunits = (prefix[e + 1] - base) / Hkv;
            const int r = pos - base;
            const int c = r / nunits, j = r - c * nunits;
            const int seg_len = min(nunits - j, pos1 - pos);
            const int b = e / S;
            int beg, end;
            clamp_range(shard_ranges[2 * e], shard_ranges[2 * e + 1], seq_lens[b], beg, end);
            const int first_page = beg >> 4, last_page = (end - 1) >> 4;
            const bool whole = (j == 0 && seg_len == nunits);
            const int slot = e * Hkv + c + (int)blockIdx.x;
            const long long row_base = (long long)b * P.max_pages_per_req;

            // table entries are fetched 32 pages (4 stages) at a time
            int tbl_page0 = 0, tbl = 0;
            for (int u = 0; ok && u < seg_len; ++u) {
                const int page0 = first_page + (j + u) * kPagesPerStage;
                const int np = min(kPagesPerStage, last_page + 1 - page0);
                if ((u & 3) == 0) {
                    tbl_page0 = page0;
                    const int lp = min(page0 + lane, last_page);
                    tbl = block_table ? block_table[row_base + lp] : (int)(row_base + lp);
                }
                const int i = lane & 7;           // page within the stage
                const int part = lane >> 3;       // 0: K lo, 1: K hi, 2: V lo, 3: V hi
                int phys = __shfl_sync(0xffffffffu, tbl, (page0 - tbl_page0) + i);
                bool bad = false;
                if (P.check_bounds && (phys < 0 || (long long)phys >= P.num_pages)) { bad = true; phys = 0; }
                const unsigned bad_mask = __ballot_sync(0xffffffffu, bad && i < np && part == 0) & 0xffu;

                if (!mbar_wait(smem_u32(&sm.empty_bar[stage]), phase ^ 1, abort_flag)) { ok = false; break; }
                const bool first = (u == 0), last = (u == seg_len - 1);
                const uint32_t full = smem_u32(&sm.full_bar[stage]);
                if (lane == 0) {
                    StageMeta mt;
                    mt.entry = e; mt.kv_head = c; mt.page0 = page0; mt.npages = np;
                    mt.tok_beg = beg; mt.tok_end = end;
                    mt.flags = (first ? kSegFirst : 0) | (last ? kSegLast : 0) | (whole ? kSegWhole : 0);
                    mt.aux = (int)bad_mask | (slot << 8);
                    sm.meta[stage] = mt;
                    mbar_arrive_expect_tx(full, (uint32_t)np * 2u * kPageBytes + (first ? (uint32_t)G * 256u : 0u));
                    if (bad_mask) atomicOr(header + kHdrStatus, kStatusBadPage);
                }
                __syncwarp();
                if (i < np) {
                    const int row = (phys * Hkv + c) * kPageSize;
                    const uint32_t dst = smem_u32(&sm.kv[stage][part >> 1][i][0]) + (part & 1) * kHalfTileBytes;
                    tma_load_2d(dst, (part >> 1) ? &v_map : &k_map, (part & 1) * 64, row, full);
                }
                if (first && lane == 0)
                    bulk_load_1d(smem_u32(&sm.q[stage][0]), q + ((size_t)b * Hq + (size_t)c * G) * kHeadDim,
                                 (uint32_t)G * 256u, full);
                ++issued;
                if (++stage == kStages) { stage = 0; phase ^= 1; }
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
            if (lane == 0) { sm.abort_flag = 1; atomicOr(header + kHdrStatus, kStatusTimeout); }
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
    const int g = lane >> 2, t = lane & 3;
    const float scale2 = P.sm_scale * 1.4426950408889634f;  // scores are kept in units of log 2
    const float kLn2 = 0.6931471805599453f;
    uint32_t qf[8][2];
    float m2[2] = {neg_inf(), neg_inf()};
    float l[2] = {0.f, 0.f};
    float acc[8][4];
    int stage = 0;
    uint32_t phase = 0, red_phase = 0;

    for (;;) {
        if (!mbar_wait(smem_u32(&sm.full_bar[stage]), phase, abort_flag)) {
            if (lane == 0) { sm.abort_flag = 1; atomicOr(header + kHdrStatus, kStatusTimeout); }
            return;
        }
        const StageMeta mt = sm.meta[stage];
        if (mt.entry < 0) return;

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

        if (warp < mt.npages) {
            const int tok0 = (mt.page0 + warp) << 4;
            int tlo = max(mt.tok_beg - tok0, 0), thi = min(mt.tok_end - tok0, kPageSize);
            if ((mt.aux >> warp) & 1) { tlo = 0; thi = 0; }
            const bool ragged = (tlo > 0) || (thi < kPageSize);
            const uint32_t k_base = smem_u32(&sm.kv[stage][0][warp][0]);
            const uint32_t v_base = smem_u32(&sm.kv[stage][1][warp][0]);

            if (ragged) {
                // tokens outside the range must contribute nothing, whatever bits they hold:
                // their value rows are cleared (0 * NaN would poison the product)
                uint8_t *vb = &sm.kv[stage][1][warp][0];
                for (int idx = lane; idx < kPageBytes / 16; idx += 32) {
                    const int row = (idx >> 3) & 15;
                    if (row < tlo || row >= thi) reinterpret_cast<uint4 *>(vb)[idx] = make_uint4(0, 0, 0, 0);
                }
                __syncwarp();
            }

            // ---- S[token, head] = K Q^T: A = K tile (row major), B = Q^T fragments
            float sc[4] = {0.f, 0.f, 0.f, 0.f};
            {
                const int row = (lane & 7) + ((lane >> 3) & 1) * 8;
                const int csel = lane >> 4;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const int chunk = 2 * ks + csel;  // 16-byte chunk of the 256-byte row
                    const uint32_t addr = k_base + (chunk >> 3) * kHalfTileBytes + row * 128 +
                                          (((chunk & 7) ^ (row & 7)) << 4);
                    uint32_t a[4];
                    ldmatrix_x4(a, addr);
                    mma_bf16(sc, a, qf[ks][0], qf[ks][1]);
                }
            }
            // sc[0],sc[1]: token g, heads 2t,2t+1;  sc[2],sc[3]: token g+8
#pragma unroll
            for (int i = 0; i < 4; ++i) sc[i] *= scale2;
            if (ragged) {
                if (g < tlo || g >= thi) { sc[0] = neg_inf(); sc[1] = neg_inf(); }
                if (g + 8 < tlo || g + 8 >= thi) { sc[2] = neg_inf(); sc[3] = neg_inf(); }
            }
            float mx0 = fmaxf(sc[0], sc[2]), mx1 = fmaxf(sc[1], sc[3]);
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
            }
            const float mn0 = fmaxf(m2[0], mx0), mn1 = fmaxf(m2[1], mx1);
            const float ms0 = (mn0 == neg_inf()) ? 0.f : mn0;  // nothing seen yet: avoid inf - inf
            const float ms1 = (mn1 == neg_inf()) ? 0.f : mn1;
            const float al0 = fast_exp2(m2[0] - ms0), al1 = fast_exp2(m2[1] - ms1);
            const float p0 = fast_exp2(sc[0] - ms0), p1 = fast_exp2(sc[1] - ms1);
            const float p2 = fast_exp2(sc[2] - ms0), p3 = fast_exp2(sc[3] - ms1);
            m2[0] = mn0; m2[1] = mn1;
            l[0] = fmaf(l[0], al0, p0 + p2);   // Z from the unrounded weights
            l[1] = fmaf(l[1], al1, p1 + p3);
            if (__any_sync(0xffffffffu, (al0 != 1.f) || (al1 != 1.f))) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    acc[i][0] *= al0; acc[i][1] *= al1; acc[i][2] *= al0; acc[i][3] *= al1;
                }
            }
            // P^T as the B operand, split into bf16 hi + lo so that the product keeps ~16 bits
            const uint32_t h0 = pack_bf16(p0, p1), h1 = pack_bf16(p2, p3);
            const uint32_t l0 = pack_bf16(p0 - bf16lo_to_f32(h0), p1 - bf16hi_to_f32(h0));
            const uint32_t l1 = pack_bf16(p2 - bf16lo_to_f32(h1), p3 - bf16hi_to_f32(h1));
            const uint32_t bh0 = movmatrix_trans(h0), bh1 = movmatrix_trans(h1);
            const uint32_t bl0 = movmatrix_trans(l0), bl1 = movmatrix_trans(l1);

            // ---- O^T[d, head] += V^T P^T: A = V^T via transposing loads
            {
                const int row = (lane & 7) + (lane >> 4) * 8;
                const int csel = (lane >> 3) & 1;
#pragma unroll
                for (int mt_i = 0; mt_i < 8; ++mt_i) {
                    const int chunk = 2 * mt_i + csel;
                    const uint32_t addr = v_base + (chunk >> 3) * kHalfTileBytes + row * 128 +
                                          (((chunk & 7) ^ (row & 7)) << 4);
                    uint32_t a[4];
                    ldmatrix_x4_trans(a, addr);
                    mma_bf16(acc[mt_i], a, bh0, bh1);
                    mma_bf16(acc[mt_i], a, bl0, bl1);
                }
            }
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
            const size_t out_row = ((size_t)mt.entry * Hq + (size_t)mt.kv_head * G);  // + head
            float *seg_slot = seg + (size_t)(mt.aux >> 8) * seg_stride;
#pragma unroll
            for (int hr = 0; hr < G / RG; ++hr) {
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
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sm.red_bar[0]));
                if (!mbar_wait(smem_u32(&sm.red_bar[0]), red_phase, abort_flag)) {
                    if (lane == 0) { sm.abort_flag = 1; atomicOr(header + kHdrStatus, kStatusTimeout); }
                    return;
                }
                for (int idx = tid; idx < RG * kHeadDim; idx += kConsumerWarps * 32) {
                    const int hl = idx >> 7, d = idx & 127;
                    const int head = hr * RG + hl;
                    float M = neg_inf();
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, sm.red_ml[w][head][0]);
                    const float Ms = (M == neg_inf()) ? 0.f : M;
                    float z = 0.f, wsum = 0.f;
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) {
                        const float ew = fast_exp2(sm.red_ml[w][head][0] - Ms);
                        z = fmaf(sm.red_ml[w][head][1], ew, z);
                        wsum = fmaf(sm.red_acc[w][hl][d], ew, wsum);
                    }
                    if (mt.flags & kSegWhole) {
                        const bool empty = (M == neg_inf());
                        o_part[(out_row + head) * kHeadDim + d] = empty ? 0.f : wsum / z;
                        if (d == 0) {
                            m_part[out_row + head] = empty ? neg_inf() : M * kLn2;
                            lse_part[out_row + head] = empty ? neg_inf() : (M + log2f(z)) * kLn2;
                        }
                    } else {
                        seg_slot[head * kHeadDim + d] = wsum;
                        if (d == 0) {
                            seg_slot[G * kHeadDim + 2 * head] = M;
                            seg_slot[G * kHeadDim + 2 * head + 1] = z;
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sm.red_bar[1]));
                if (!mbar_wait(smem_u32(&sm.red_bar[1]), red_phase, abort_flag)) {
                    if (lane == 0) { sm.abort_flag = 1; atomicOr(header + kHdrStatus, kStatusTimeout); }
                    return;
                }
                red_phase ^= 1;
            }
        }
        if (++stage == kStages) { stage = 0; phase ^= 1; }
    }
}

// ------------------------------------------------------------------ merge kernel
// One CTA per (request, shard, KV head); thread = channel.  Merges the segment
// states a (shard, KV head) was split into by CTA-slice boundaries, and writes
// the empty-shard convention (o = 0, m = lse = -inf).
template <int G>
__global__ void __launch_bounds__(kHeadDim)
merge_kernel(const int *__restrict__ header, const int *__restrict__ prefix, const float *__restrict__ seg,
             int seg_stride, float *__restrict__ o_part, float *__restrict__ m_part,
             float *__restrict__ lse_part, int num_q_heads, int num_kv_heads)
{
    const int c = blockIdx.x;
    const int e = blockIdx.y;
    const int d = threadIdx.x;
    const float kLn2 = 0.6931471805599453f;
    const int base = prefix[e];
    const int cnt = prefix[e + 1] - base;
    const size_t out_row = (size_t)e * num_q_heads + (size_t)c * G;
    if (cnt == 0) {
#pragma unroll
        for (int h = 0; h < G; ++h) {
            o_part[(out_row + h) * kHeadDim + d] = 0.f;
            if (d == 0) { m_part[out_row + h] = neg_inf(); lse_part[out_row + h] = neg_inf(); }
        }
        return;
    }
    const int nunits = cnt / num_kv_heads;
    const int per_cta = header[kHdrUnitsPerCta];
    const int p0 = base + c * nunits, p1 = p0 + nunits;
    const int first = p0 / per_cta, last = (p1 - 1) / per_cta;
    if (first == last) return;  // the sweep wrote this state directly
    const int unit = e * num_kv_heads + c;
#pragma unroll
    for (int h = 0; h < G; ++h) {
        float M = neg_inf();
        for (int i = first; i <= last; ++i)
            M = fmaxf(M, seg[(size_t)(unit + i) * seg_stride + G * kHeadDim + 2 * h]);
        const bool empty = (M == neg_inf());
        const float Ms = empty ? 0.f : M;
        float z = 0.f, wsum = 0.f;
        for (int i = first; i <= last; ++i) {
            const float *sl = seg + (size_t)(unit + i) * seg_stride;
            const float ew = fast_exp2(sl[G * kHeadDim + 2 * h] - Ms);
            z = fmaf(sl[G * kHeadDim + 2 * h + 1], ew, z);
            wsum = fmaf(sl[h * kHeadDim + d], ew, wsum);
        }
        o_part[(out_row + h) * kHeadDim + d] = empty ? 0.f : wsum / z;
        if (d == 0) {
            m_part[out_row + h] = empty ? neg_inf() : M * kLn2;
            lse_part[out_row + h] = empty ? neg_inf() : (M + log2f(z)) * kLn2;
        }
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// A [rows, 128] bf16 view of a KV pool, boxes of 16 rows x 64 channels, 128B swizzle.
inline int make_pool_map(CUtensorMap *out, const void *pool, long long num_pages, int num_kv_heads, char *msg,
                         size_t msg_len)
{
    static EncodeTiledFn encode = nullptr;
    static std::mutex mu;
    struct Entry { const void *pool; long long pages; int heads; CUtensorMap map; };
    static Entry cache[16];
    static int n_cached = 0, next = 0;
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < n_cached; ++i)
        if (cache[i].pool == pool && cache[i].pages == num_pages && cache[i].heads == num_kv_heads) {
            *out = cache[i].map;
            return 0;
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
    const cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)num_pages * num_kv_heads * kPageSize};
    const cuuint64_t strides[1] = {(cuuint64_t)kHeadDim * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kPageSize};
    const cuuint32_t estr[2] = {1, 1};
    CUtensorMap map;
    CUresult r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(pool), dims, strides, box,
                        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(msg, msg_len, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return -1;
    }
    Entry &slot = cache[next];
    slot.pool = pool; slot.pages = num_pages; slot.heads = num_kv_heads; slot.map = map;
    next = (next + 1) % 16;
    if (n_cached < 16) ++n_cached;
    *out = map;
    return 0;
}

template <int G>
int launch_sweep_g(const CUtensorMap &kmap, const CUtensorMap &vmap, const void *q, const int32_t *bt,
                   const int32_t *sl, const int32_t *sr, float *o, float *m, float *l, const DevParams &P,
                   char *ws, const WorkspaceLayout &wsl, int n_ctas, cudaStream_t st, cudaEvent_t ev0,
                   cudaEvent_t ev1, char *msg, size_t msg_len, int *launches)
{
    int *header = reinterpret_cast<int *>(ws + wsl.header_off);
    int *prefix = reinterpret_cast<int *>(ws + wsl.prefix_off);
    float *seg = reinterpret_cast<float *>(ws + wsl.seg_off);
    const int n_entries = P.batch * P.max_shards;
    const size_t smem = sizeof(SweepSmem<G>) + 1024;
    static bool attr_set[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set[dev & 63]) {
        cudaError_t e = cudaFuncSetAttribute(sweep_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) { snprintf(msg, msg_len, "cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return -5; }
        attr_set[dev & 63] = true;
    }
    plan_kernel<<<1, 1024, 0, st>>>(sl, sr, header, prefix, n_entries, P.max_shards, P.num_kv_heads, n_ctas);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { snprintf(msg, msg_len, "plan_kernel launch: %s", cudaGetErrorString(e)); return -5; }
    if (ev0) cudaEventRecord(ev0, st);
    sweep_kernel<G><<<n_ctas, kSweepThreads, smem, st>>>(kmap, vmap, (const uint16_t *)q, bt, sl, sr, o, m, l,
                                                          header, prefix, seg, wsl.seg_stride, P);
    e = cudaGetLastError();
    if (ev1) cudaEventRecord(ev1, st);
    if (e != cudaSuccess) { snprintf(msg, msg_len, "sweep_kernel launch: %s", cudaGetErrorString(e)); return -5; }
    dim3 mgrid(P.num_kv_heads, n_entries);
    merge_kernel<G><<<mgrid, kHeadDim, 0, st>>>(header, prefix, seg, wsl.seg_stride, o, m, l, P.num_q_heads,
                                                P.num_kv_heads);
    e = cudaGetLastError();
    if (e != cudaSuccess) { snprintf(msg, msg_len, "merge_kernel launch: %s", cudaGetErrorString(e)); return -5; }
    *launches = 3;
    return 0;
}

inline int launch_sweep(const void *q, const void *k_cache, const void *v_cache, const int32_t *bt,
                        const int32_t *sl, const int32_t *sr, float *o, float *m, float *l, const DevParams &P,
                        char *ws, const WorkspaceLayout &wsl, int sm_count, cudaStream_t st, cudaEvent_t ev0,
                        cudaEvent_t ev1, char *msg, size_t msg_len, int *launches)
{
    CUtensorMap kmap, vmap;
    if (make_pool_map(&kmap, k_cache, P.num_pages, P.num_kv_heads, msg, msg_len)) return -5;
    if (make_pool_map(&vmap, v_cache, P.num_pages, P.num_kv_heads, msg, msg_len)) return -5;
    const int n_ctas = sm_count < kMaxSweepCtas ? sm_count : kMaxSweepCtas;
    switch (P.group) {
    case 1: return launch_sweep_g<1>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, st, ev0, ev1, msg, msg_len, launches);
    case 2: return launch_sweep_g<2>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, st, ev0, ev1, msg, msg_len, launches);
    case 4: return launch_sweep_g<4>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, st, ev0, ev1, msg, msg_len, launches);
    default: return launch_sweep_g<8>(kmap, vmap, q, bt, sl, sr, o, m, l, P, ws, wsl, n_ctas, st, ev0, ev1, msg, msg_len, launches);
    }
}

}  // namespace qf
