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
//   * K is split eight ways over a thread-block cluster, so a 2,560 x 4,096 weight keeps 160 CTAs busy;
//     a CTA's whole weight slice (128 x K/8 bf16) is requested by TMA at the very start of the kernel,
//     before the programmatic dependency on the previous kernel is waited for (weights are never
//     produced on the path), and is consumed box by box as it lands.
//   * the eight partial tiles are summed over distributed shared memory in rank order (bit-deterministic),
//     each rank finishing 16 of the tile's 128 output features.
//
// Stage 0 (W_o): X = bf16(a), epilogue u' = bf16(z + Y), plus each tile's sum of squares of the rounded
// stream per request.  Stage 1 (W_q): X = bf16(g u' / sqrt(mean u'^2 + eps)) built in the prologue from
// stage 0's outputs, epilogue q = bf16(Y).
//
// Every wait on an mbarrier is bounded; a wait that runs out raises the CTA's abort flag and a status bit,
// the CTA stops computing but still takes part in the cluster barriers, drains its copies and frees its
// tensor memory.  No TMA multicast is used.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

#include "qf_common.cuh"
#include "qf_page_math.cuh"

namespace qf {

constexpr int kProjThreads   = 128;   // thread t owns accumulator row t (one output feature)
constexpr int kProjTileOut   = 128;   // output features per CTA = rows of the tensor-core tile
constexpr int kProjSplits    = 8;     // K splits = CTAs of a cluster
constexpr int kProjBoxK      = 64;    // bf16 per TMA box row: 128 bytes, one swizzle span
constexpr int kProjMaxBoxes  = 10;    // K / 8 / 64 <= 10, i.e. K <= 5,120
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
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar,
                                            unsigned long long policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar), "l"(policy) : "memory");
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

// Dynamic shared memory: this header (1 KB), then n_boxes weight boxes [128 rows][128 B], then n_boxes
// activation boxes [NP rows][128 B]; every box is 1,024-byte aligned.  The partial tile [NP][128] fp32
// reuses the weight boxes once the products are done (the host checks that it fits).
struct ProjSmemHeader {
    alignas(8) unsigned long long w_full[kProjMaxBoxes];
    alignas(8) unsigned long long mma_done;
    uint32_t tmem_base;
    int abort_flag;
    float ssq[kProjMaxBatch];      // stage 0: this rank's sums of squares; stage 1: 1/rms per request
    float half_sum[kProjMaxBatch]; // stage 1 prologue
};
static_assert(sizeof(ProjSmemHeader) <= 1024, "header must fit its kilobyte");
constexpr int kProjWBoxBytes = kProjTileOut * 128;
inline size_t proj_smem_bytes(int n_boxes, int np)
{
    return 1024 /* alignment slack */ + 1024 + (size_t)n_boxes * (kProjWBoxBytes + np * 128);
}

template <int STAGE, int NP>
__global__ void __launch_bounds__(kProjThreads, 1)
proj_kernel(const __grid_constant__ CUtensorMap w_map, ProjArgs A)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem_al = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    ProjSmemHeader &sm = *reinterpret_cast<ProjSmemHeader *>(smem_al);
    const int tid = threadIdx.x, warp = tid >> 5;
    const int rank = (int)cluster_rank();                 // which eighth of K
    const int tile = (int)blockIdx.x / kProjSplits;       // which 128 output features
    const int k_slice = A.k_total / kProjSplits, n_boxes = k_slice / kProjBoxK;
    uint8_t *w_boxes = smem_al + 1024;                    // [n_boxes][128][128 B]
    uint8_t *x_boxes = w_boxes + (size_t)n_boxes * kProjWBoxBytes;   // [n_boxes][NP][128 B]
    const int k0 = rank * k_slice;
    volatile int *abort_flag = &sm.abort_flag;

    if (tid == 0) {
        for (int i = 0; i < n_boxes; ++i) mbar_init(smem_u32(&sm.w_full[i]), 1);
        mbar_init(smem_u32(&sm.mma_done), 1);
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // the whole weight slice, now: it does not depend on anything the stream computed before
        const unsigned long long policy = l2_evict_first_policy();
        for (int i = 0; i < n_boxes; ++i) {
            mbar_arrive_expect_tx(smem_u32(&sm.w_full[i]), kProjTileOut * 128);
            tma_load_2d(smem_u32(w_boxes + (size_t)i * kProjWBoxBytes), &w_map, k0 + i * kProjBoxK, tile * kProjTileOut, smem_u32(&sm.w_full[i]), policy);
        }
    }
    if (warp == 0) tmem_alloc(smem_u32(&sm.tmem_base), 64);

    grid_dependency_wait();     // everything below reads what earlier kernels of the stream wrote
    grid_launch_dependents();
    if (STAGE == 0 && blockIdx.x == 0 && tid == 0) *A.status = 0u;

    // ---- activations of this K slice, as the B operand: [NP rows][k_slice] bf16, 128B-swizzled boxes
    if (STAGE == 1) {
        // 1/rms per request from stage 0's per-tile sums of squares, summed in tile order (two interleaved halves)
        const int n = tid & (kProjMaxBatch - 1), half = tid / kProjMaxBatch;
        float s = 0.f;
        if (n < A.batch)
            for (int p = half; p < A.ssq_tiles; p += 2) s += ld_sync_f32(A.ssq_part + (size_t)p * kProjMaxBatch + n);
        if (half == 1) sm.half_sum[n] = s;
        __syncthreads();
        if (half == 0) sm.ssq[n] = 1.0f / sqrtf((s + sm.half_sum[n]) * A.inv_d_model + A.eps);
        __syncthreads();
    }
    {
        const int chunks_per_row = k_slice / 8;           // 16-byte chunks of 8 bf16
        for (int idx = tid; idx < NP * chunks_per_row; idx += kProjThreads) {
            const int m = idx / chunks_per_row, ck = idx - m * chunks_per_row;
            const int k = ck * 8, box = k / kProjBoxK, c = (k % kProjBoxK) / 8;
            uint4 pk = make_uint4(0u, 0u, 0u, 0u);
            if (m < A.batch) {
                if (STAGE == 0) {
                    const float4 lo = *reinterpret_cast<const float4 *>(A.a + (size_t)m * A.k_total + k0 + k);
                    const float4 hi = *reinterpret_cast<const float4 *>(A.a + (size_t)m * A.k_total + k0 + k + 4);
                    pk = make_uint4(pack_bf16(lo.x, lo.y), pack_bf16(lo.z, lo.w), pack_bf16(hi.x, hi.y), pack_bf16(hi.z, hi.w));
                } else {
                    const uint4 uw = *reinterpret_cast<const uint4 *>(A.u_in + (size_t)m * A.k_total + k0 + k);
                    const uint4 gw = *reinterpret_cast<const uint4 *>(A.g + k0 + k);
                    const float r = sm.ssq[m];
                    const uint32_t uu[4] = {uw.x, uw.y, uw.z, uw.w}, gg[4] = {gw.x, gw.y, gw.z, gw.w};
                    uint32_t o[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)   // g*u is exact in fp32 (two bf16 factors); one rounding by r, one to bf16
                        o[e] = pack_bf16(bf16lo_to_f32(gg[e]) * bf16lo_to_f32(uu[e]) * r,
                                         bf16hi_to_f32(gg[e]) * bf16hi_to_f32(uu[e]) * r);
                    pk = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
            *reinterpret_cast<uint4 *>(x_boxes + (size_t)box * (NP * 128) + m * 128 + ((c ^ (m & 7)) * 16)) = pk;
        }
    }
    // the tensor core reads shared memory through the async proxy: make the stores above visible to it
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(&sm.tmem_base);

    // ---- products: one thread issues them box by box as the weight lands
    if (tid == 32) {
        constexpr uint32_t idesc = umma_idesc_bf16(NP);
        bool ok = true;
        for (int i = 0; i < n_boxes && ok; ++i) {
            if (!mbar_wait(smem_u32(&sm.w_full[i]), 0, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint64_t ad = umma_desc_k_sw128(smem_u32(w_boxes + (size_t)i * kProjWBoxBytes));
            const uint64_t bd = umma_desc_k_sw128(smem_u32(x_boxes + (size_t)i * (NP * 128)));
#pragma unroll
            for (int kk = 0; kk < kProjBoxK / 16; ++kk)   // 16 bf16 = 32 bytes = 2 descriptor units along K
                umma_bf16(tmem, ad + 2 * kk, bd + 2 * kk, idesc, (i | kk) ? 1u : 0u);
        }
        if (ok) {
            umma_commit(smem_u32(&sm.mma_done));
        } else {
            sm.abort_flag = 1;
            atomicOr(A.status, (unsigned)kStatusTimeout);
            // copies still in flight must land before this CTA's shared memory goes away
            for (int i = 0; i < n_boxes; ++i)
                for (unsigned it = 0; it < (1u << 20); ++it)
                    if (mbar_try_wait(smem_u32(&sm.w_full[i]), 0)) break;
            mbar_arrive(smem_u32(&sm.mma_done));
        }
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
        const int j = tid & (kProjRowsPerRank - 1), n0 = tid / kProjRowsPerRank;   // feature within the rank's 16, request lane
        const int o = tile * kProjTileOut + rank * kProjRowsPerRank + j;
        const uint32_t part_addr = smem_u32(part);
#pragma unroll
        for (int i = 0; i < NP / 8; ++i) {
            const int n = n0 + 8 * i;
            float y = 0.f;
#pragma unroll
            for (int c = 0; c < kProjSplits; ++c)
                y += ld_peer_f32(part_addr + (uint32_t)((n * kProjTileOut + rank * kProjRowsPerRank + j) * 4), (uint32_t)c);
            float sq = 0.f;
            if (n < A.batch) {
                if (STAGE == 0) {
                    const float zf = __uint_as_float((uint32_t)A.z[(size_t)n * A.n_out + o] << 16);
                    const __nv_bfloat16 ub = __float2bfloat16_rn(zf + y);
                    A.out[(size_t)n * A.n_out + o] = *reinterpret_cast<const uint16_t *>(&ub);
                    const float uf = __bfloat162float(ub);
                    sq = uf * uf;
                } else {
                    const __nv_bfloat16 qb = __float2bfloat16_rn(y);
                    A.out[(size_t)n * A.n_out + o] = *reinterpret_cast<const uint16_t *>(&qb);
                }
            }
            if (STAGE == 0) {
                // sum of squares over the rank's 16 features: the 16 lanes of a half warp, fixed tree
#pragma unroll
                for (int off = 8; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
                if (j == 0) sm.ssq[n] = sq;
            }
        }
    }
    cluster_sync_all();          // partial tiles are no longer read; stage 0: every rank's sums of squares are in place
    if (STAGE == 0) {
        if (rank == 0 && tid < NP) {
            float s = 0.f;
            const uint32_t addr = smem_u32(&sm.ssq[tid]);
#pragma unroll
            for (int c = 0; c < kProjSplits; ++c) s += ld_peer_f32(addr, (uint32_t)c);
            A.ssq_part[(size_t)tile * kProjMaxBatch + tid] = (tid < A.batch) ? s : 0.f;
        }
        cluster_sync_all();      // nobody leaves while rank 0 still reads its shared memory
    }
    if (warp == 0) tmem_dealloc(tmem, 64);
}

// ------------------------------------------------------------------ host side
// A [rows][cols] row-major bf16 weight as 128B-swizzled boxes of 128 rows x 64 columns.
inline int make_weight_map(CUtensorMap *out, const void *w, int rows, int cols, char *msg, size_t msg_len)
{
    typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                 const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    static std::mutex mu;
    struct Entry { const void *w; int rows, cols; CUtensorMap map; };
    static Entry cache[32];
    static int n_cached = 0, next = 0;
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < n_cached; ++i)
        if (cache[i].w == w && cache[i].rows == rows && cache[i].cols == cols) {
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
        encode = (EncodeFn)fn;
    }
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kProjBoxK, (cuuint32_t)kProjTileOut};
    const cuuint32_t estr[2] = {1, 1};
    CUtensorMap map;
    CUresult r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(w), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(msg, msg_len, "cuTensorMapEncodeTiled (weight) failed with CUresult %d", (int)r);
        return -1;
    }
    Entry &slot = cache[next];
    slot.w = w; slot.rows = rows; slot.cols = cols; slot.map = map;
    next = (next + 1) % 32;
    if (n_cached < 32) ++n_cached;
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
    if ((size_t)np * kProjTileOut * 4 > (size_t)n_boxes * kProjWBoxBytes) return false;   // partial tile reuses the weight boxes
    return proj_smem_bytes(n_boxes, np) <= 227 * 1024;
}

template <int STAGE, int NP>
cudaError_t launch_proj_np(const CUtensorMap &map, const ProjArgs &args, cudaStream_t st)
{
    const int n_boxes = args.k_total / (kProjSplits * kProjBoxK);
    const size_t smem = proj_smem_bytes(n_boxes, NP);
    cudaError_t e = cudaFuncSetAttribute(proj_kernel<STAGE, NP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(args.n_out / kProjTileOut * kProjSplits));
    cfg.blockDim = dim3(kProjThreads);
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
    return cudaLaunchKernelEx(&cfg, proj_kernel<STAGE, NP>, map, args);
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
