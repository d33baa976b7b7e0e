// The cache side's projection pair at a layer boundary (Section 4: the cache side holds W_q and W_o;
// a stage ends in u' = z + W_o a and the next one opens with q = W_q N_1(u'); appendix "The cache side
// must batch": the products run over the co-resident requests of a batch).
//
// Both products are skinny: a few requests (at most 64 here) against a weight matrix of tens of
// megabytes that is read exactly once.  They are bound by streaming the weight, so the kernel is built
// around that stream and the tensor cores only have to keep out of its way:
//
//   * Y^T[out x batch] = W[out x K] . X^T[K x batch]: the weight is the M-side operand of
//     tcgen05.mma (128 output features per CTA), the batch is the N side (16..64 columns), the
//     accumulator lives in tensor memory.
//   * K is split eight ways over a thread-block cluster, so a 2,560 x 4,096 weight keeps 160 CTAs busy.
//     A CTA's weight slice (128 x K/8 bf16) arrives in TMA requests of several adjacent 128-row x 128-byte
//     boxes.  How many bytes a request reads contiguously per weight row decides what the stream reaches
//     (one 128-byte box per request: a third of the HBM rate; 512 bytes per row: more than twice that),
//     so a request is as large as shared memory allows and the ring is as deep as what is left (often one
//     slot).  The first requests go out at the very start of the kernel, before the programmatic dependency
//     on the previous kernel is waited for (weights are never produced on the path); a slot is refilled as
//     soon as the products that read it have completed (tcgen05.commit on the slot's barrier).  The ring,
//     not the whole slice, is resident so that two CTAs fit an SM and every cluster of a product is resident
//     at once: with the whole slice resident the kernel ran in two waves and took twice as long.
//   * 256 threads stage the activation slice (the 128 that own accumulator rows plus four helper warps).
//   * the eight partial tiles are summed over distributed shared memory in rank order (bit-deterministic),
//     each rank finishing 16 of the tile's 128 output features; two cluster barriers in all.
//
// Stage 0 (W_o): X = bf16(a), epilogue u' = bf16(z + Y), plus each tile's sum of squares of the rounded
// stream per request.  Stage 1 (W_q): X = bf16(g u' / sqrt(mean u'^2 + eps)) built in the prologue from
// stage 0's outputs, epilogue q = bf16(Y).
//
// Every wait on an mbarrier is bounded; a wait that runs out raises the CTA's abort flag and a status bit,
// the CTA stops computing but still takes part in the cluster barriers, drains its copies and frees its
// tensor memory.  Every TMA load lands in the shared memory of the CTA that issued it.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

#include "qf_common.cuh"
#include "qf_page_math.cuh"

namespace qf {

constexpr int kProjThreads   = 128;   // thread t owns accumulator row t (one output feature)
constexpr int kProjCtaThreads = 256;  // the CTA: those 128 plus four warps that only help stage the activations
constexpr int kProjTileOut   = 128;   // output features per CTA = rows of the tensor-core tile
constexpr int kProjSplits    = 8;     // K splits = CTAs of a cluster
constexpr int kProjBoxK      = 64;    // bf16 per TMA box row: 128 bytes, one swizzle span
constexpr int kProjMaxBoxes  = 10;    // K / 8 / 64 <= 10, i.e. K <= 5,120
constexpr int kProjMaxRing   = 4;     // weight requests in flight per CTA, at most
constexpr int kProjMaxBatch  = 64;
constexpr int kProjRowsPerRank = kProjTileOut / kProjSplits;   // 16

struct ProjArgs {
    const float *a;            // stage 0: [batch][K] fp32
    const uint16_t *u_in;      // stage 1: [batch][K] bf16 (stage 0's output)
    const uint16_t *g;         // stage 1: [K] bf16
    const uint16_t *z;         // stage 0: [batch][n_out] bf16
    uint16_t *out;             // [batch][n_out] bf16 (u' or q)
    float *ssq_part;           // [tiles of stage 0][kProjMaxBatch]: stage 0 writes, stage 1 reads
    unsigned *status;          // bit 1 (QF_STATUS_TIMEOUT) is ORed in when a wait runs out
    int batch, n_out, k_total;
    int ssq_tiles;             // stage 1: number of stage 0 tiles
    int ring_sb, ring_slots;   // boxes per TMA request, requests in flight per CTA (proj_ring)
    float inv_d_model, eps;    // stage 1
};

// ---- tcgen05 / cluster PTX
__device__ __forceinline__ void tmem_alloc(uint32_t holder_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem] . B[smem]^T, 128 x N x 16, bf16 in, fp32 out
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 16 consecutive accumulator columns of this thread's row
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16])
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ float ld_peer_f32(uint32_t local_smem_addr, uint32_t rank)
{
    uint32_t ra;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_smem_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(ra) : "memory");
    return v;
}
// One request: `sb` adjacent boxes (the map's box is [sb column blocks][128 rows][64 bf16]) starting at weight
// row `row` and column block `kblock`; they land as sb consecutive swizzled [128][128 B] tiles.
__device__ __forceinline__ void st_peer_f32(uint32_t local_smem_addr, uint32_t rank, float v)
{
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_smem_addr), "r"(rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(ra), "f"(v) : "memory");
}
__device__ __forceinline__ void tma_load_boxes(uint32_t dst, const CUtensorMap *map, int row, int kblock, uint32_t bar,
                                               unsigned long long policy)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(dst), "l"(map), "r"(0), "r"(row), "r"(kblock), "r"(bar), "l"(policy) : "memory");
}

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes, 128B-swizzled, eight-row
// groups 1,024 bytes apart (what a TMA box of 64 bf16 per row leaves): start address, leading offset 1
// (unused for swizzled K-major), stride offset 1,024 B, descriptor version 1, layout type 2 (128B swizzle).
__device__ __forceinline__ uint64_t umma_desc_k_sw128(uint32_t smem_addr)
{
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// Dynamic shared memory: this header (5 KB), then a ring of weight boxes [128 rows][128 B], then n_boxes
// activation boxes [NP rows][128 B]; every box is 1,024-byte aligned.  The partial tile [NP][128] fp32
// reuses the ring once the products are done (the host checks that it fits).
struct ProjSmemHeader {
    alignas(8) unsigned long long w_full[kProjMaxRing];    // a slot's box has landed
    alignas(8) unsigned long long w_empty[kProjMaxRing];   // the products reading a slot have completed
    alignas(8) unsigned long long mma_done;
    uint32_t tmem_base;
    int abort_flag;
    float ssq[kProjMaxBatch];      // stage 0: this rank's sums of squares; stage 1: 1/rms per request
    float part_sum[3][kProjMaxBatch];   // stage 1 prologue
    float ssq_recv[kProjSplits][kProjMaxBatch];   // stage 0, rank 0: every rank's sums of squares, pushed by their owners
    alignas(16) uint16_t gain[kProjMaxBoxes * kProjBoxK];   // stage 1: this K slice of g
};
constexpr int kProjHeaderBytes = 5120;
static_assert(sizeof(ProjSmemHeader) <= kProjHeaderBytes, "header must fit its five kilobytes");
constexpr int kProjWBoxBytes = kProjTileOut * 128;
inline size_t proj_smem_bytes(int ring, int n_boxes, int np)
{
    return 1024 /* alignment slack */ + kProjHeaderBytes + (size_t)ring * kProjWBoxBytes + (size_t)n_boxes * np * 128;
}
// The ring: `slots` requests in flight, each of `sb` adjacent boxes (sb divides the slice's box count).
// Preferred: the largest request that still leaves room for two CTAs per SM (then every cluster of a product
// is resident at once), and only then as many slots as fit: the bytes a request reads contiguously per weight
// row matter more than the ring's depth (one 512-byte-per-row request at a time beat two 256-byte ones in
// flight).  The ring must also hold the partial tile.  Falls back to one CTA per SM when nothing smaller fits.
struct ProjRing { int sb, slots; };
inline ProjRing proj_ring(int n_boxes, int np)
{
    const int need = (np * kProjTileOut * 4 + kProjWBoxBytes - 1) / kProjWBoxBytes;   // boxes the partial tile covers
    for (int pass = 0; pass < 2; ++pass) {
        const size_t budget = (pass == 0 ? 113 : 227) * 1024;
        for (int sb = n_boxes; sb >= 1; --sb) {
            if (n_boxes % sb) continue;
            const int n_req = n_boxes / sb;
            for (int slots = (n_req < kProjMaxRing ? n_req : kProjMaxRing); slots >= 1; --slots) {
                if (sb * slots < need) break;
                if (proj_smem_bytes(sb * slots, n_boxes, np) <= budget) return ProjRing{sb, slots};
            }
        }
    }
    return ProjRing{0, 0};
}

template <int STAGE, int NP>
__global__ void __launch_bounds__(kProjCtaThreads, 2)
proj_kernel(const __grid_constant__ CUtensorMap w_map, ProjArgs A)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem_al = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    ProjSmemHeader &sm = *reinterpret_cast<ProjSmemHeader *>(smem_al);
    const int tid = threadIdx.x, warp = tid >> 5;
    const bool is_main = tid < kProjThreads;   // the helper warps leave after the staging (they still join the cluster barriers)
    const int rank = (int)cluster_rank();                 // which eighth of K
    const int tile = (int)blockIdx.x / kProjSplits;       // which 128 output features
    const int k_slice = A.k_total / kProjSplits, n_boxes = k_slice / kProjBoxK;
    const int sb = A.ring_sb, slots = A.ring_slots, n_req = n_boxes / sb;   // boxes per request, requests in flight, requests
    uint8_t *w_boxes = smem_al + kProjHeaderBytes;        // [slots][sb][128][128 B]
    uint8_t *x_boxes = w_boxes + (size_t)slots * sb * kProjWBoxBytes;   // [n_boxes][NP][128 B]
    const int k0 = rank * k_slice;
    volatile int *abort_flag = &sm.abort_flag;

    // thread 32 owns the weight stream and the products
    const unsigned long long policy = l2_evict_first_policy();
    auto issue_req = [&](int r) {   // request r: boxes [r sb, r sb + sb) of this CTA's slice
        const int slot = r % slots;
        mbar_arrive_expect_tx(smem_u32(&sm.w_full[slot]), (uint32_t)sb * kProjWBoxBytes);
        tma_load_boxes(smem_u32(w_boxes + (size_t)slot * sb * kProjWBoxBytes), &w_map, tile * kProjTileOut,
                       k0 / kProjBoxK + r * sb, smem_u32(&sm.w_full[slot]), policy);
    };
    int issued = 0;
    if (tid == 32) {
        for (int i = 0; i < slots; ++i) {
            mbar_init(smem_u32(&sm.w_full[i]), 1);
            mbar_init(smem_u32(&sm.w_empty[i]), 1);
        }
        mbar_init(smem_u32(&sm.mma_done), 1);
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // the first fill of the ring, now: the weight does not depend on anything the stream computed before
        for (; issued < slots; ++issued) issue_req(issued);
    }
    if (warp == 0) tmem_alloc(smem_u32(&sm.tmem_base), 64);

    grid_dependency_wait();     // everything below reads what earlier kernels of the stream wrote
    grid_launch_dependents();
    if (STAGE == 0 && blockIdx.x == 0 && tid == 0) *A.status = 0u;

    // ---- activations of this K slice, as the B operand: [NP rows][k_slice] bf16, 128B-swizzled boxes.
    // Global loads are issued eight items at a time per thread before any of them is used (the prologue is
    // a few dependent round trips to L2 long; done one by one it was longer than streaming the weight).
    constexpr int kU = 8;
    const int chunks_per_row = k_slice / 8;               // 16-byte chunks of 8 bf16
    const int n_items = A.batch * chunks_per_row;         // rows at or beyond the batch are zero-filled below
    auto item_addr = [&](int idx, int &m, int &k) { m = idx / chunks_per_row; k = (idx - m * chunks_per_row) * 8; };
    auto x_slot = [&](int m, int k) -> uint4 * {
        const int box = k / kProjBoxK, c = (k % kProjBoxK) / 8;
        return reinterpret_cast<uint4 *>(x_boxes + (size_t)box * (NP * 128) + m * 128 + ((c ^ (m & 7)) * 16));
    };
    // what the epilogue adds to the product (stage 0), fetched now so that it has long arrived by then
    const int ep_j = tid & (kProjRowsPerRank - 1), ep_n0 = tid / kProjRowsPerRank;
    const int ep_o = tile * kProjTileOut + rank * kProjRowsPerRank + ep_j;
    uint16_t zreg[NP / 8];
#pragma unroll
    for (int i = 0; i < NP / 8; ++i) {
        const int n = ep_n0 + 8 * i;
        zreg[i] = (STAGE == 0 && is_main && n < A.batch) ? A.z[(size_t)n * A.n_out + ep_o] : (uint16_t)0;
    }
    if (STAGE == 0) {
        for (int base = tid; base < n_items; base += kProjCtaThreads * kU) {
            float4 lo[kU], hi[kU];
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const int idx = base + u * kProjCtaThreads;
                if (idx < n_items) {
                    int m, k;
                    item_addr(idx, m, k);
                    const float *src = A.a + (size_t)m * A.k_total + k0 + k;
                    lo[u] = *reinterpret_cast<const float4 *>(src);
                    hi[u] = *reinterpret_cast<const float4 *>(src + 4);
                }
            }
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const int idx = base + u * kProjCtaThreads;
                if (idx < n_items) {
                    int m, k;
                    item_addr(idx, m, k);
                    *x_slot(m, k) = make_uint4(pack_bf16(lo[u].x, lo[u].y), pack_bf16(lo[u].z, lo[u].w),
                                               pack_bf16(hi[u].x, hi[u].y), pack_bf16(hi[u].z, hi[u].w));
                }
            }
        }
    } else {
        // the gain slice and the first batch of the stream go out before the sums of squares are waited for
        for (int i = tid; i < k_slice / 8; i += kProjCtaThreads)
            reinterpret_cast<uint4 *>(sm.gain)[i] = *reinterpret_cast<const uint4 *>(A.g + k0 + i * 8);
        uint4 uw[kU];
        auto load_batch = [&](int base) {
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const int idx = base + u * kProjCtaThreads;
                if (idx < n_items) {
                    int m, k;
                    item_addr(idx, m, k);
                    uw[u] = *reinterpret_cast<const uint4 *>(A.u_in + (size_t)m * A.k_total + k0 + k);
                }
            }
        };
        load_batch(tid);
        {
            // 1/rms per request from stage 0's per-tile sums of squares: four interleaved quarters of the tiles, each
            // summed in tile order, then added in quarter order
            const int n = tid & (kProjMaxBatch - 1), quarter = tid / kProjMaxBatch;
            float s = 0.f;
            if (n < A.batch) {
                for (int p0 = quarter; p0 < A.ssq_tiles; p0 += 4 * kU) {
                    float v[kU];
#pragma unroll
                    for (int u = 0; u < kU; ++u) {
                        const int p = p0 + 4 * u;
                        v[u] = (p < A.ssq_tiles) ? ld_sync_f32(A.ssq_part + (size_t)p * kProjMaxBatch + n) : 0.f;
                    }
#pragma unroll
                    for (int u = 0; u < kU; ++u) s += v[u];
                }
            }
            if (quarter > 0) sm.part_sum[quarter - 1][n] = s;
            __syncthreads();
            if (quarter == 0)
                sm.ssq[n] = 1.0f / sqrtf((((s + sm.part_sum[0][n]) + sm.part_sum[1][n]) + sm.part_sum[2][n]) * A.inv_d_model + A.eps);
            __syncthreads();
        }
        for (int base = tid; base < n_items; base += kProjCtaThreads * kU) {
            if (base != tid) load_batch(base);
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const int idx = base + u * kProjCtaThreads;
                if (idx < n_items) {
                    int m, k;
                    item_addr(idx, m, k);
                    const uint4 gw = *reinterpret_cast<const uint4 *>(sm.gain + k);
                    const float r = sm.ssq[m];
                    const uint32_t uu[4] = {uw[u].x, uw[u].y, uw[u].z, uw[u].w}, gg[4] = {gw.x, gw.y, gw.z, gw.w};
                    uint32_t o[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)   // g*u is exact in fp32 (two bf16 factors); one rounding by r, one to bf16
                        o[e] = pack_bf16(bf16lo_to_f32(gg[e]) * bf16lo_to_f32(uu[e]) * r,
                                         bf16hi_to_f32(gg[e]) * bf16hi_to_f32(uu[e]) * r);
                    *x_slot(m, k) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
        }
    }
    for (int idx = n_items + tid; idx < NP * chunks_per_row; idx += kProjCtaThreads) {   // padding rows
        int m, k;
        item_addr(idx, m, k);
        *x_slot(m, k) = make_uint4(0u, 0u, 0u, 0u);
    }
    // the tensor core reads shared memory through the async proxy: make the stores above visible to it
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(&sm.tmem_base);

    // ---- products: thread 32 issues them box by box as the weight lands, and refills the slots behind them
    if (tid == 32) {
        constexpr uint32_t idesc = umma_idesc_bf16(NP);
        bool ok = true;
        int consumed = 0;
        for (int r = 0; r < n_req && ok; ++r) {
            // keep the ring full: the slot of the next request to issue was last used by request (issued - slots),
            // whose products must have completed (tcgen05.commit on the slot's barrier) before it is overwritten
            while (issued < n_req && issued < r + slots) {
                const int prev = issued - slots;
                if (prev >= 0 &&
                    !mbar_wait(smem_u32(&sm.w_empty[prev % slots]), (uint32_t)((prev / slots) & 1), abort_flag)) { ok = false; break; }
                issue_req(issued++);
            }
            if (!ok) break;
            const int slot = r % slots;
            if (!mbar_wait(smem_u32(&sm.w_full[slot]), (uint32_t)((r / slots) & 1), abort_flag)) { ok = false; break; }
            consumed = r + 1;
            tc_fence_after();
            for (int j = 0; j < sb; ++j) {
                const int i = r * sb + j;     // box of the slice
                const uint64_t ad = umma_desc_k_sw128(smem_u32(w_boxes + (size_t)(slot * sb + j) * kProjWBoxBytes));
                const uint64_t bd = umma_desc_k_sw128(smem_u32(x_boxes + (size_t)i * (NP * 128)));
#pragma unroll
                for (int kk = 0; kk < kProjBoxK / 16; ++kk)   // 16 bf16 = 32 bytes = 2 descriptor units along K
                    umma_bf16(tmem, ad + 2 * kk, bd + 2 * kk, idesc, (i | kk) ? 1u : 0u);
            }
            umma_commit(smem_u32(&sm.w_empty[slot]));     // arrives when the products above have completed
        }
        if (ok) {
            umma_commit(smem_u32(&sm.mma_done));
        } else {
            sm.abort_flag = 1;
            atomicOr(A.status, (unsigned)kStatusTimeout);
            // copies still in flight must land before this CTA's shared memory goes away
            for (int r = consumed; r < issued; ++r)
                for (unsigned it = 0; it < (1u << 20); ++it)
                    if (mbar_try_wait(smem_u32(&sm.w_full[r % slots]), (uint32_t)((r / slots) & 1))) break;
            mbar_arrive(smem_u32(&sm.mma_done));
        }
    }
    if (!is_main) {   // helper warps: nothing left to do but keep the cluster barriers' counts whole
        cluster_sync_all();
        cluster_sync_all();
        return;
    }
    const bool done = mbar_wait(smem_u32(&sm.mma_done), 0, abort_flag) && !*abort_flag;
    if (!done && tid == 0) { sm.abort_flag = 1; atomicOr(A.status, (unsigned)kStatusTimeout); }
    tc_fence_after();

    // ---- this CTA's partial tile: accumulator row t, NP columns -> shared memory [n][128]
    float *part = reinterpret_cast<float *>(w_boxes);
#pragma unroll
    for (int c16 = 0; c16 < NP / 16; ++c16) {
        float v[16];
        if (done) {
            tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(c16 * 16), v);
        } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = 0.f;
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) part[(c16 * 16 + i) * kProjTileOut + tid] = v[i];
    }
    tc_fence_before();
    cluster_sync_all();          // every rank's partial tile is in place

    // ---- sum the eight partials in rank order; this rank finishes output features [16 rank, 16 rank + 16)
    {
        const uint32_t part_addr = smem_u32(part);
        float pv[NP / 8][kProjSplits];
#pragma unroll
        for (int i = 0; i < NP / 8; ++i)        // every remote read is issued before any is summed
#pragma unroll
            for (int c = 0; c < kProjSplits; ++c)
                pv[i][c] = ld_peer_f32(part_addr + (uint32_t)(((ep_n0 + 8 * i) * kProjTileOut + rank * kProjRowsPerRank + ep_j) * 4),
                                       (uint32_t)c);
#pragma unroll
        for (int i = 0; i < NP / 8; ++i) {
            const int n = ep_n0 + 8 * i;
            float y = 0.f;
#pragma unroll
            for (int c = 0; c < kProjSplits; ++c) y += pv[i][c];
            float sq = 0.f;
            if (n < A.batch) {
                if (STAGE == 0) {
                    const float zf = __uint_as_float((uint32_t)zreg[i] << 16);
                    const __nv_bfloat16 ub = __float2bfloat16_rn(zf + y);
                    A.out[(size_t)n * A.n_out + ep_o] = *reinterpret_cast<const uint16_t *>(&ub);
                    const float uf = __bfloat162float(ub);
                    sq = uf * uf;
                } else {
                    const __nv_bfloat16 qb = __float2bfloat16_rn(y);
                    A.out[(size_t)n * A.n_out + ep_o] = *reinterpret_cast<const uint16_t *>(&qb);
                }
            }
            if (STAGE == 0) {
                // sum of squares over the rank's 16 features: the 16 lanes of a half warp, fixed tree
#pragma unroll
                for (int off = 8; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
                if (ep_j == 0) st_peer_f32(smem_u32(&sm.ssq_recv[rank][n]), 0u, sq);   // into rank 0's shared memory
            }
        }
    }
    // Partial tiles are no longer read by anybody, and (stage 0) every rank's sums of squares have arrived in
    // rank 0's shared memory: after this barrier a CTA touches only its own shared memory, so it may leave.
    cluster_sync_all();
    if (STAGE == 0 && rank == 0 && tid < NP) {
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < kProjSplits; ++c) s += sm.ssq_recv[c][tid];
        A.ssq_part[(size_t)tile * kProjMaxBatch + tid] = (tid < A.batch) ? s : 0.f;
    }
    if (warp == 0) tmem_dealloc(tmem, 64);
}

// ------------------------------------------------------------------ host side
// A [rows][cols] row-major bf16 weight seen as [cols / 64 column blocks][rows][64]: a box is sb adjacent column
// blocks of 128 rows, each landing as a 128B-swizzled [128][128 B] tile.
inline int make_weight_map(CUtensorMap *out, const void *w, int rows, int cols, int sb, char *msg, size_t msg_len)
{
    typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                 const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    static std::mutex mu;
    struct Entry { const void *w; int rows, cols, sb; CUtensorMap map; };
    // One descriptor per (pointer, shape, request size), hashed by the pointer: a decode loop walks every layer's
    // weights each step, so the cache holds a whole model's worth and a lookup is a handful of probes.
    constexpr int kCacheEntries = 1024, kProbes = 8;
    static Entry cache[kCacheEntries];   // zero-initialised: w == nullptr marks a free entry
    const size_t home = (size_t)(((uintptr_t)w >> 8) * 0x9E3779B97F4A7C15ull >> 40) % kCacheEntries;
    std::lock_guard<std::mutex> lock(mu);
    size_t victim = home;
    for (int i = 0; i < kProbes; ++i) {
        Entry &c = cache[(home + i) % kCacheEntries];
        if (c.w == w && c.rows == rows && c.cols == cols && c.sb == sb) {
            *out = c.map;
            return 0;
        }
        if (c.w == nullptr) { victim = (home + i) % kCacheEntries; break; }
    }
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
            snprintf(msg, msg_len, "cuTensorMapEncodeTiled entry point not available");
            return -1;
        }
        encode = (EncodeFn)fn;
    }
    const cuuint64_t dims[3] = {(cuuint64_t)kProjBoxK, (cuuint64_t)rows, (cuuint64_t)(cols / kProjBoxK)};
    const cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)kProjBoxK * 2};
    const cuuint32_t box[3] = {(cuuint32_t)kProjBoxK, (cuuint32_t)kProjTileOut, (cuuint32_t)sb};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUtensorMap map;
    CUresult r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(w), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(msg, msg_len, "cuTensorMapEncodeTiled (weight) failed with CUresult %d", (int)r);
        return -1;
    }
    Entry &slot = cache[victim];   // a free entry among the probes, else the home entry is replaced
    slot.w = w; slot.rows = rows; slot.cols = cols; slot.sb = sb; slot.map = map;
    *out = map;
    return 0;
}

// Padded batch (columns of the tensor-core tile): the next multiple of 16.
inline int proj_padded_batch(int batch) { return (batch + 15) / 16 * 16; }

// Can one product [n_out x k_total] with this batch run?  (shape rules and the shared-memory budget)
inline bool proj_shape_ok(int batch, int n_out, int k_total)
{
    if (batch < 1 || batch > kProjMaxBatch || n_out < kProjTileOut || n_out % kProjTileOut) return false;
    if (k_total % (kProjSplits * kProjBoxK) || k_total / (kProjSplits * kProjBoxK) > kProjMaxBoxes) return false;
    const int np = proj_padded_batch(batch), n_boxes = k_total / (kProjSplits * kProjBoxK);
    return proj_ring(n_boxes, np).slots > 0;
}

template <int STAGE, int NP>
cudaError_t launch_proj_np(const CUtensorMap &map, const ProjArgs &args, cudaStream_t st)
{
    const int n_boxes = args.k_total / (kProjSplits * kProjBoxK);
    const ProjRing ring = proj_ring(n_boxes, NP);
    ProjArgs a2 = args;
    a2.ring_sb = ring.sb;
    a2.ring_slots = ring.slots;
    const size_t smem = proj_smem_bytes(ring.sb * ring.slots, n_boxes, NP);
    // the attribute is raised once per device to the largest footprint this instantiation can have
    static bool attr_set[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set[dev & 63]) {
        cudaError_t ea = cudaFuncSetAttribute(proj_kernel<STAGE, NP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              227 * 1024);
        if (ea != cudaSuccess) return ea;
        attr_set[dev & 63] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(args.n_out / kProjTileOut * kProjSplits));
    cfg.blockDim = dim3(kProjCtaThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kProjSplits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, proj_kernel<STAGE, NP>, map, a2);
}
template <int STAGE>
cudaError_t launch_proj(const CUtensorMap &map, const ProjArgs &args, cudaStream_t st)
{
    switch (proj_padded_batch(args.batch)) {
    case 16: return launch_proj_np<STAGE, 16>(map, args, st);
    case 32: return launch_proj_np<STAGE, 32>(map, args, st);
    case 48: return launch_proj_np<STAGE, 48>(map, args, st);
    default: return launch_proj_np<STAGE, 64>(map, args, st);
    }
}

}  // namespace qf
