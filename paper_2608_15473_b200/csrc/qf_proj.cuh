// The cache side's projection pair at a layer boundary (Section 4: the cache side holds W_q and W_o;
// a stage ends in u' = z + W_o a and the next one opens with q = W_q N_1(u'); the appendix paragraph on
// batching at the cache side: the products run over the co-resident requests of a batch).
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
//   * split-K sum over distributed shared memory: rank r finishes requests n = 8 i + r.  Every rank sends
//     accumulator row t, column n, straight from tensor memory into rank (n mod 8)'s receive area with stores
//     that count their bytes on a transaction barrier of the receiver, which then adds the eight partials in
//     rank order (bit-deterministic).  One cluster barrier in all, with a relaxed arrival: it only says that
//     a rank is running (or, for large batches whose receive area reuses the ring, that its products are done).
//
// Stage 0 (W_o): X = bf16(a), epilogue u' = bf16(z + Y), plus each tile's sum of squares of the rounded
// stream per request.  Stage 1 (W_q): X = bf16(g u' / sqrt(mean u'^2 + eps)) built in the prologue from
// stage 0's outputs, epilogue q = bf16(Y).
//
// Every wait on an mbarrier is bounded; a wait that runs out raises the CTA's abort flag and a status bit,
// the CTA stops computing but still takes part in the cluster barrier, sends (zeros) what its peers count on,
// drains its copies and frees its tensor memory.  Every TMA load lands in the shared memory of the CTA that
// issued it.
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

struct ProjArgs {
    const float *a;            // stage 0: [batch][K] fp32
    const uint16_t *u_in;      // stage 1: [batch][K] bf16 (stage 0's output)
    const uint16_t *g;         // stage 1: [K] bf16
    const uint16_t *z;         // stage 0: [batch][n_out] bf16
    uint16_t *out;             // [batch][n_out] bf16 (u' or q)
    float *ssq_part;           // [tiles of stage 0][kProjMaxBatch]: stage 0 writes, stage 1 reads
    unsigned long long *status; // tagged status word (proj_status_or): QF_STATUS_TIMEOUT is ORed in when a wait runs out
    int batch, n_out, k_total;
    int ssq_tiles;             // stage 1: number of stage 0 tiles
    int ring_sb, ring_slots;   // boxes per TMA request, requests in flight per CTA (proj_ring)
    int recv_aliased;          // the split-K receive area reuses the ring (large batches) instead of its own room
    float inv_d_model, eps;    // stage 1
};

// The pair's status word is STICKY: bits stay until the host reads them (qf_project_status reads and clears),
// so a failure in one layer's pair is not wiped by the next layer's, nor by a later replay of a captured graph.
// The workspace is never assumed initialised: a word counts only if its upper 56 bits carry this tag, anything
// else reads as "clean".
constexpr unsigned long long kProjStatusTag = 0x51F1A7C0DE5EEDull;   // 56 bits
__device__ __forceinline__ void proj_status_or(unsigned long long *w, unsigned bits)
{
    unsigned long long old = *reinterpret_cast<volatile unsigned long long *>(w);
    for (int tries = 0; tries < (1 << 12); ++tries) {
        const unsigned long long cur = ((old >> 8) == kProjStatusTag) ? (old & 0xffull) : 0ull;
        const unsigned long long prev = atomicCAS(w, old, (kProjStatusTag << 8) | cur | bits);
        if (prev == old) return;
        old = prev;
    }
}

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
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// The address, in the cluster's shared window, of CTA `rank`'s copy of one of this CTA's shared-memory locations.
__device__ __forceinline__ uint32_t peer_addr(uint32_t local_smem_addr, uint32_t rank)
{
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_smem_addr), "r"(rank));
    return ra;
}
// Store into a peer's shared memory that counts its four bytes on a transaction barrier of that same peer: the
// receiver learns that the data has landed from its own barrier, without a cluster-wide release and acquire.
__device__ __forceinline__ void st_async_f32(uint32_t cluster_addr, float v, uint32_t cluster_mbar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];"
                 ::"r"(cluster_addr), "f"(v), "r"(cluster_mbar) : "memory");
}
// One request: `sb` adjacent boxes (the map's box is [sb column blocks][128 rows][64 bf16]) starting at weight
// row `row` and column block `kblock`; they land as sb consecutive swizzled [128][128 B] tiles.
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

// Dynamic shared memory: this header (5 KB), then (small batches) the split-K receive area
// [8 source ranks][NP / 8 requests][128 features] fp32, then a ring of weight boxes [128 rows][128 B], then
// n_boxes activation boxes [NP rows][128 B]; every box is 1,024-byte aligned.  For large batches the receive
// area has no room of its own and reuses the ring once every rank's products are done (the host checks that it fits).
struct ProjSmemHeader {
    alignas(8) unsigned long long w_full[kProjMaxRing];    // a slot's box has landed
    alignas(8) unsigned long long w_empty[kProjMaxRing];   // the products reading a slot have completed
    alignas(8) unsigned long long mma_done;
    alignas(8) unsigned long long recv_full;               // every rank's rows of this rank's requests have landed
    uint32_t tmem_base;
    int abort_flag;
    float ssq[kProjMaxBatch];      // stage 0: this rank's sums of squares; stage 1: 1/rms per request
    float part_sum[3][kProjMaxBatch];   // stage 1 prologue
    float ssq_warp[4][kProjMaxBatch / kProjSplits];   // stage 0: per-warp sums of squares of this rank's requests
    alignas(16) uint16_t gain[kProjMaxBoxes * kProjBoxK];   // stage 1: this K slice of g
};
constexpr int kProjHeaderBytes = 5120;
static_assert(sizeof(ProjSmemHeader) <= kProjHeaderBytes, "header must fit its five kilobytes");
constexpr int kProjWBoxBytes = kProjTileOut * 128;
__host__ __device__ constexpr int proj_recv_bytes(int np) { return kProjSplits * (np / kProjSplits) * kProjTileOut * 4; }
inline size_t proj_smem_bytes(int ring, int n_boxes, int np, bool own_recv)
{
    return 1024 /* alignment slack */ + kProjHeaderBytes + (own_recv ? proj_recv_bytes(np) : 0) +
           (size_t)ring * kProjWBoxBytes + (size_t)n_boxes * np * 128;
}
// The ring: `slots` requests in flight, each of `sb` adjacent boxes (sb divides the slice's box count).
// Preferred: the largest request that still leaves room for two CTAs per SM (then every cluster of a product
// is resident at once), and only then as many slots as fit: the bytes a request reads contiguously per weight
// row matter more than the ring's depth (one 512-byte-per-row request at a time beat two 256-byte ones in
// flight).  Falls back to one CTA per SM when nothing smaller fits.  The split-K receive area gets room of its
// own (one cluster barrier fewer) when that costs the ring nothing; otherwise it reuses the ring, which must
// then be large enough for it.
struct ProjRing { int sb, slots; bool own_recv; };
inline ProjRing proj_ring_for(int n_boxes, int np, bool own_recv, size_t budget)
{
    const int need = own_recv ? 0 : (proj_recv_bytes(np) + kProjWBoxBytes - 1) / kProjWBoxBytes;
    for (int sb = n_boxes; sb >= 1; --sb) {
        if (n_boxes % sb) continue;
        const int n_req = n_boxes / sb;
        for (int slots = (n_req < kProjMaxRing ? n_req : kProjMaxRing); slots >= 1; --slots) {
            if (sb * slots < need) break;
            if (proj_smem_bytes(sb * slots, n_boxes, np, own_recv) <= budget) return ProjRing{sb, slots, own_recv};
        }
    }
    return ProjRing{0, 0, own_recv};
}
inline ProjRing proj_ring(int n_boxes, int np)
{
    for (int pass = 0; pass < 2; ++pass) {
        const size_t budget = (pass == 0 ? 113 : 227) * 1024;
        const ProjRing shared = proj_ring_for(n_boxes, np, false, budget), own = proj_ring_for(n_boxes, np, true, budget);
        if (own.slots > 0 && own.sb >= shared.sb && own.sb * own.slots >= shared.sb * shared.slots) return own;
        if (shared.slots > 0) return shared;
    }
    return ProjRing{0, 0, false};
}

template <int STAGE, int NP>
__global__ void __launch_bounds__(kProjCtaThreads, 2)
proj_kernel(const __grid_constant__ CUtensorMap w_map, ProjArgs A)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem_al = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    ProjSmemHeader &sm = *reinterpret_cast<ProjSmemHeader *>(smem_al);
    const int tid = threadIdx.x, warp = tid >> 5;
    const bool is_main = tid < kProjThreads;   // the helper warps leave after the staging (they still join the cluster barrier)
    const int rank = (int)cluster_rank();                 // which eighth of K
    const int tile = (int)blockIdx.x / kProjSplits;       // which 128 output features
    const int k_slice = A.k_total / kProjSplits, n_boxes = k_slice / kProjBoxK;
    const int sb = A.ring_sb, slots = A.ring_slots, n_req = n_boxes / sb;   // boxes per request, requests in flight, requests
    const bool recv_aliased = A.recv_aliased != 0;
    constexpr int kCols = NP / kProjSplits;               // requests this rank finishes: n = i * 8 + rank, i < kCols
    uint8_t *w_boxes = smem_al + kProjHeaderBytes + (recv_aliased ? 0 : proj_recv_bytes(NP));   // [slots][sb][128][128 B]
    float *recv = reinterpret_cast<float *>(recv_aliased ? w_boxes : smem_al + kProjHeaderBytes);   // [8 sources][kCols][128]
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
        mbar_init(smem_u32(&sm.recv_full), 1);
        mbar_arrive_expect_tx(smem_u32(&sm.recv_full), (uint32_t)proj_recv_bytes(NP));   // what the eight ranks will send
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // the first fill of the ring, now: the weight does not depend on anything the stream computed before
        for (; issued < slots; ++issued) issue_req(issued);
    }
    if (warp == 0) tmem_alloc(smem_u32(&sm.tmem_base), 64);

    grid_dependency_wait();     // everything below reads what earlier kernels of the stream wrote
    grid_launch_dependents();

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
    const int ep_o = tile * kProjTileOut + (tid & (kProjTileOut - 1));   // this thread's output feature
    uint16_t zreg[kCols];
#pragma unroll
    for (int i = 0; i < kCols; ++i) {
        const int n = i * kProjSplits + rank;
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
    // With a receive area of its own a rank may be written by its peers as soon as it runs and its barriers are
    // initialised: this arrival, waited for only just before the first remote store, says so.  It orders no data
    // (relaxed: a releasing arrival cost a microsecond here, and at the top of the kernel so did a relaxed one,
    // while the cluster's CTAs were still being placed).
    if (!recv_aliased) cluster_arrive_relaxed();
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
            proj_status_or(A.status, (unsigned)kStatusTimeout);
            // copies still in flight must land before this CTA's shared memory goes away
            for (int r = consumed; r < issued; ++r)
                for (unsigned it = 0; it < (1u << 20); ++it)
                    if (mbar_try_wait(smem_u32(&sm.w_full[r % slots]), (uint32_t)((r / slots) & 1))) break;
            mbar_arrive(smem_u32(&sm.mma_done));
        }
    }
    if (!is_main) {   // helper warps: nothing left to do but keep the cluster barrier's count whole
        if (recv_aliased) cluster_arrive_relaxed();
        cluster_wait();
        return;
    }
    const bool done = mbar_wait(smem_u32(&sm.mma_done), 0, abort_flag) && !*abort_flag;
    if (!done && tid == 0) { sm.abort_flag = 1; proj_status_or(A.status, (unsigned)kStatusTimeout); }
    tc_fence_after();

    // ---- split-K sum.  Rank r finishes requests n = 8 i + r (all 128 features of each): every rank sends
    // accumulator row t, column n, straight from tensor memory into recv[its own rank][i][t] of rank n mod 8,
    // with stores that count their bytes on the receiver's transaction barrier.  The one cluster barrier comes
    // first: with its own receive area a rank can be written as soon as it runs (it arrived after its staging);
    // a receive area inside the ring can be written once the rank's products are done, which this thread has
    // seen on mma_done before it arrives (the arrival carries no data, so it need not release anything).
    if (recv_aliased) cluster_arrive_relaxed();
    cluster_wait();
    {
        const uint32_t mine = smem_u32(recv + (size_t)(rank * kCols) * kProjTileOut + tid);
        const uint32_t bar = smem_u32(&sm.recv_full);
        uint32_t dst[kProjSplits], dst_bar[kProjSplits];
#pragma unroll
        for (int r = 0; r < kProjSplits; ++r) {
            dst[r] = peer_addr(mine, (uint32_t)r);
            dst_bar[r] = peer_addr(bar, (uint32_t)r);
        }
#pragma unroll
        for (int c16 = 0; c16 < NP / 16; ++c16) {
            float v[16];
            if (done) {
                tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(c16 * 16), v);
            } else {      // a rank that gave up still sends (zeros): its peers count on the bytes
#pragma unroll
                for (int k = 0; k < 16; ++k) v[k] = 0.f;
            }
#pragma unroll
            for (int k = 0; k < 16; ++k)   // column n = 16 c16 + k: request i = n / 8 of rank n mod 8
                st_async_f32(dst[k & 7] + (uint32_t)((2 * c16 + (k >> 3)) * kProjTileOut * 4), v[k], dst_bar[k & 7]);
        }
    }
    tc_fence_before();
    // Wait for what the eight ranks send here.  The limit is twice any other wait's, and a local abort does not cut
    // it short: a peer that gives up elsewhere still sends, and this CTA must not leave while stores are on their way.
    {
        bool landed = false;
        for (unsigned it = 0; it < 2u * kSpinLimit && !landed; ++it) {
            landed = mbar_try_wait(smem_u32(&sm.recv_full), 0u);
            if (!landed && it > 64) __nanosleep(64);
        }
        if (!landed && tid == 0) proj_status_or(A.status, (unsigned)kStatusTimeout);
    }

    // ---- the eight partials of this rank's requests, summed in rank order, and the epilogue
    float sq[kCols];
#pragma unroll
    for (int i = 0; i < kCols; ++i) {
        const int n = i * kProjSplits + rank;
        float pv[kProjSplits];
#pragma unroll
        for (int c = 0; c < kProjSplits; ++c) pv[c] = recv[(size_t)(c * kCols + i) * kProjTileOut + tid];
        float y = 0.f;
#pragma unroll
        for (int c = 0; c < kProjSplits; ++c) y += pv[c];
        sq[i] = 0.f;
        if (n < A.batch) {
            if (STAGE == 0) {
                const float zf = __uint_as_float((uint32_t)zreg[i] << 16);
                const __nv_bfloat16 ub = __float2bfloat16_rn(zf + y);
                A.out[(size_t)n * A.n_out + ep_o] = *reinterpret_cast<const uint16_t *>(&ub);
                const float uf = __bfloat162float(ub);
                sq[i] = uf * uf;
            } else {
                const __nv_bfloat16 qb = __float2bfloat16_rn(y);
                A.out[(size_t)n * A.n_out + ep_o] = *reinterpret_cast<const uint16_t *>(&qb);
            }
        }
    }
    if (STAGE == 0) {
        // sums of squares of the rounded stream over the tile's 128 features, per request: a fixed tree inside
        // each warp, then the four warps in order
#pragma unroll
        for (int i = 0; i < kCols; ++i) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) sq[i] += __shfl_xor_sync(0xffffffffu, sq[i], off);
            if ((tid & 31) == 0) sm.ssq_warp[warp][i] = sq[i];
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kProjThreads) : "memory");   // the 128 main threads (the helpers have left)
        if (tid < kCols) {
            const int n = tid * kProjSplits + rank;
            const float s4 = ((sm.ssq_warp[0][tid] + sm.ssq_warp[1][tid]) + sm.ssq_warp[2][tid]) + sm.ssq_warp[3][tid];
            A.ssq_part[(size_t)tile * kProjMaxBatch + n] = (n < A.batch) ? s4 : 0.f;
        }
    }
    // every warp's reads of tensor memory are complete (they preceded its stores, which have all landed here)
    asm volatile("bar.sync 1, %0;" ::"n"(kProjThreads) : "memory");
    tc_fence_after();
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
    a2.recv_aliased = ring.own_recv ? 0 : 1;
    const size_t smem = proj_smem_bytes(ring.sb * ring.slots, n_boxes, NP, ring.own_recv);
    // the attribute is raised once per device to the largest footprint this instantiation can have
    {
        static std::mutex attr_mu;   // any host thread may be the first on a device
        static bool attr_set[64];
        int dev = 0;
        cudaGetDevice(&dev);
        std::lock_guard<std::mutex> lock(attr_mu);
        if (!attr_set[dev & 63]) {
            cudaError_t ea = cudaFuncSetAttribute(proj_kernel<STAGE, NP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                  227 * 1024);
            if (ea != cudaSuccess) return ea;
            attr_set[dev & 63] = true;
        }
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
