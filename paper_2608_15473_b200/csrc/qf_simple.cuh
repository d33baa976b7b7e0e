// Plain-load sweep kernel: one CTA per (request, KV head, shard), no staging,
// no tensor cores.  It exists as a validation aid for the staged kernel (it is
// selected by QF_FLAG_SIMPLE_KERNEL); it follows the same online-softmax
// recurrence (Section 5: (W, Z) add over disjoint sets) warp by warp.
#pragma once

#include "qf_common.cuh"

namespace qf {

constexpr int kSimpleWarps = 8;

template <int G>
__global__ void __launch_bounds__(kSimpleWarps * 32)
sweep_simple_kernel(const uint16_t *__restrict__ q, const uint16_t *__restrict__ k_cache,
                    const uint16_t *__restrict__ v_cache, const int *__restrict__ block_table,
                    const int *__restrict__ seq_lens, const int *__restrict__ shard_ranges,
                    float *__restrict__ o_part, float *__restrict__ m_part, float *__restrict__ lse_part,
                    DevParams P, unsigned long long *header, unsigned long long epoch)
{
    const int s = blockIdx.x, c = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = P.max_shards, Hq = P.num_q_heads, Hkv = P.num_kv_heads;

    if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0) header[kHdrLastEpoch] = epoch;

    int beg, end;
    const int max_tokens = P.max_tokens;
    clamp_range(shard_ranges[(b * S + s) * 2], shard_ranges[(b * S + s) * 2 + 1], seq_lens[b], max_tokens, beg, end);
    if (P.check_bounds && seq_lens[b] > max_tokens && s == 0 && c == 0 && threadIdx.x == 0)
        epoch_or(header + kHdrStatus, epoch, kStatusBadPage);   // a length the block-table row cannot address

    // lane owns channels [4*lane, 4*lane+4) of every vector
    float qr[G][4];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const uint2 w = *reinterpret_cast<const uint2 *>(q + ((size_t)b * Hq + c * G + g) * kHeadDim + lane * 4);
        qr[g][0] = bf16lo_to_f32(w.x); qr[g][1] = bf16hi_to_f32(w.x);
        qr[g][2] = bf16lo_to_f32(w.y); qr[g][3] = bf16hi_to_f32(w.y);
    }

    float m[G], l[G], acc[G][4];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m[g] = neg_inf(); l[g] = 0.f;
        acc[g][0] = acc[g][1] = acc[g][2] = acc[g][3] = 0.f;
    }

    for (int i = beg + warp; i < end; i += kSimpleWarps) {
        const int lp = i >> 4, slot = i & 15;
        long long phys = block_table ? (long long)block_table[(size_t)b * P.max_pages_per_req + lp]
                                     : (long long)b * P.max_pages_per_req + lp;
        if (P.check_bounds && (phys < 0 || phys >= P.num_pages)) {
            if (lane == 0) epoch_or(header + kHdrStatus, epoch, kStatusBadPage);
            continue;
        }
        const size_t row = kv_row_offset(P, phys, c, slot) + lane * 4;
        const uint2 kw = *reinterpret_cast<const uint2 *>(k_cache + row);
        const uint2 vw = *reinterpret_cast<const uint2 *>(v_cache + row);
        const float k0 = bf16lo_to_f32(kw.x), k1 = bf16hi_to_f32(kw.x);
        const float k2 = bf16lo_to_f32(kw.y), k3 = bf16hi_to_f32(kw.y);
        const float v0 = bf16lo_to_f32(vw.x), v1 = bf16hi_to_f32(vw.x);
        const float v2 = bf16lo_to_f32(vw.y), v3 = bf16hi_to_f32(vw.y);
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float d = qr[g][0] * k0;
            d = fmaf(qr[g][1], k1, d);
            d = fmaf(qr[g][2], k2, d);
            d = fmaf(qr[g][3], k3, d);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
            const float sc = d * P.sm_scale;
            const float mn = fmaxf(m[g], sc);
            const float alpha = __expf(m[g] - mn);   // m = -inf on the first token: e^{-inf} = 0
            const float p = __expf(sc - mn);
            l[g] = l[g] * alpha + p;
            acc[g][0] = fmaf(p, v0, acc[g][0] * alpha);
            acc[g][1] = fmaf(p, v1, acc[g][1] * alpha);
            acc[g][2] = fmaf(p, v2, acc[g][2] * alpha);
            acc[g][3] = fmaf(p, v3, acc[g][3] * alpha);
            m[g] = mn;
        }
    }

    // merge the warps' states (same (W, Z) algebra), normalise, write
    __shared__ float sm_m[kSimpleWarps][G];
    __shared__ float sm_l[kSimpleWarps][G];
    __shared__ float sm_acc[kSimpleWarps][G][kHeadDim];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        if (lane == 0) { sm_m[warp][g] = m[g]; sm_l[warp][g] = l[g]; }
        *reinterpret_cast<float4 *>(&sm_acc[warp][g][lane * 4]) =
            make_float4(acc[g][0], acc[g][1], acc[g][2], acc[g][3]);
    }
    __syncthreads();

    for (int idx = threadIdx.x; idx < G * kHeadDim; idx += kSimpleWarps * 32) {
        const int g = idx / kHeadDim, d = idx % kHeadDim;
        float M = neg_inf();
#pragma unroll
        for (int w = 0; w < kSimpleWarps; ++w) M = fmaxf(M, sm_m[w][g]);
        const size_t slot = out_entry(P, b * S + s) * Hq + c * G + g;
        if (M == neg_inf()) {  // empty shard
            o_part[slot * kHeadDim + d] = 0.f;
            if (d == 0) { m_part[slot] = neg_inf(); lse_part[slot] = neg_inf(); }
            continue;
        }
        float z = 0.f, wsum = 0.f;
#pragma unroll
        for (int w = 0; w < kSimpleWarps; ++w) {
            if (sm_m[w][g] == neg_inf()) continue;
            const float e = __expf(sm_m[w][g] - M);
            z = fmaf(sm_l[w][g], e, z);
            wsum = fmaf(sm_acc[w][g][d], e, wsum);
        }
        o_part[slot * kHeadDim + d] = wsum / z;
        if (d == 0) { m_part[slot] = M; lse_part[slot] = M + logf(z); }
    }
}

}  // namespace qf
