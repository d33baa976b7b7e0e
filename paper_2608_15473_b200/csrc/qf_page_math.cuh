// Shared-memory / tensor-core building blocks of the sweep kernels (sm_100a).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include "qf_common.cuh"

namespace qf {

constexpr unsigned kSpinLimit = 1u << 24;

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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          unsigned limit = kSpinLimit)
{
    for (unsigned it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 64) {
            if (*abort_flag) return false;
            __nanosleep(64);
        }
    }
    return false;
}
// L2 policy for the K/V stream: every byte is used once, so its lines should be the first to go and
// leave the L2 to what is reused (shard states, segment slots, block table, q).
__device__ __forceinline__ unsigned long long l2_evict_first_policy()
{
    unsigned long long policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
// One TMA box (a page of one KV head: 64 channels x 16 rows x 2 halves = 4 KB; or of eight heads: 32 KB).
__device__ __forceinline__ void tma_load_page(uint32_t dst, const CUtensorMap *map, int row, uint32_t bar,
                                              unsigned long long policy)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(dst), "l"(map), "r"(0), "r"(row), "r"(0), "r"(bar), "l"(policy) : "memory");
}
// The same box from a token-major pool: 16 rows of one KV head, Hkv rows apart (a 4-D view: channel half,
// KV head, token, half of the row).
__device__ __forceinline__ void tma_load_page_nhd(uint32_t dst, const CUtensorMap *map, int kv_head, int token_row,
                                                  uint32_t bar, unsigned long long policy)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %4, %5}], [%6], %7;"
        ::"r"(dst), "l"(map), "r"(0), "r"(kv_head), "r"(token_row), "r"(0), "r"(bar), "l"(policy) : "memory");
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


// One page (16 tokens of one KV head) against the G query heads of its group: the online-softmax
// step of Section 5 ((W, Z) add over disjoint sets) on tensor cores.
//
//   k_base, v_base  shared-memory addresses of the page's K and V tiles; a tile is two half tiles
//                   ([16 rows][128 B], channels 0-63 and 64-127, 128B-swizzled), half_stride apart
//   [tlo, thi)      rows of the page inside the shard's token range (ragged = not all 16)
//   qf              Q^T fragments (B operand), zero for heads >= G
//   m2, l, acc      running max (log-2 units), running Z (this thread's rows), O^T accumulators
//                   for heads 2t, 2t+1 of the lane (t = lane & 3)
//
// Fragment maps (m16n8k16): S = K Q^T has tokens on M and heads on N; P is re-laid out as the B
// operand of O^T += V^T P^T with an in-register 8x8 transpose; Z uses the unrounded weights and
// P is split into bf16 hi + lo so the product keeps about 16 bits.
__device__ __forceinline__ void process_page(uint32_t k_base, uint32_t v_base, int half_stride, int tlo, int thi,
                                             bool ragged, const uint32_t (&qf)[8][2], float (&m2)[2],
                                             float (&l)[2], float (&acc)[8][4], float scale2, int lane)
{
    const int g = lane >> 2;
    if (ragged) {
        // tokens outside the range must contribute nothing, whatever bits they hold:
        // their value rows are cleared (0 * NaN would poison the product)
        for (int idx = lane; idx < kPageBytes / 16; idx += 32) {
            const int row = (idx >> 3) & 15;
            if (row < tlo || row >= thi) {
                const uint32_t addr = v_base + (idx >> 7) * half_stride + (idx & 127) * 16;
                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0) : "memory");
            }
        }
        __syncwarp();
    }

    // ---- S[token, head] = K Q^T: A = K tile (row major), B = Q^T fragments
    // All K fragments are fetched before the first MMA, and the V fragments right after the last one, so
    // that shared-memory latency overlaps the tensor pipe and the softmax arithmetic below.
    float sc[4] = {0.f, 0.f, 0.f, 0.f};
    uint32_t vfrag[8][4];
    {
        float sc_odd[4] = {0.f, 0.f, 0.f, 0.f};  // two accumulators: half the dependent-MMA chain
        uint32_t kfrag[8][4];
        const int row = (lane & 7) + ((lane >> 3) & 1) * 8;
        const int csel = lane >> 4;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const int chunk = 2 * ks + csel;  // 16-byte chunk of the 256-byte row
            ldmatrix_x4(kfrag[ks], k_base + (chunk >> 3) * half_stride + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
        }
#pragma unroll
        for (int ks = 0; ks < 8; ks += 2) {
            mma_bf16(sc, kfrag[ks], qf[ks][0], qf[ks][1]);
            mma_bf16(sc_odd, kfrag[ks + 1], qf[ks + 1][0], qf[ks + 1][1]);
        }
        const int vrow = (lane & 7) + (lane >> 4) * 8;
        const int vsel = (lane >> 3) & 1;
#pragma unroll
        for (int mt_i = 0; mt_i < 8; ++mt_i) {   // A = V^T via transposing loads
            const int chunk = 2 * mt_i + vsel;
            ldmatrix_x4_trans(vfrag[mt_i],
                              v_base + (chunk >> 3) * half_stride + vrow * 128 + (((chunk & 7) ^ (vrow & 7)) << 4));
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) sc[i] += sc_odd[i];
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

    // ---- O^T[d, head] += V^T P^T: the eight hi products first, then the eight lo products, so that no
    // MMA waits on the one just issued for the same accumulator
#pragma unroll
    for (int mt_i = 0; mt_i < 8; ++mt_i) mma_bf16(acc[mt_i], vfrag[mt_i], bh0, bh1);
#pragma unroll
    for (int mt_i = 0; mt_i < 8; ++mt_i) mma_bf16(acc[mt_i], vfrag[mt_i], bl0, bl1);
}

}  // namespace qf
