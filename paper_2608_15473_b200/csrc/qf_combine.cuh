// Merge of shard states (Section 5): n-way, overflow-safe form of the pairwise
// lerp / sigma / logaddexp combine.  One warp per (request, query head); each
// lane owns four channels, so a shard's 512-byte vector is one coalesced read.
#pragma once

#include "qf_common.cuh"

namespace qf {

constexpr int kCombineWarps = 4;

__global__ void __launch_bounds__(kCombineWarps * 32)
combine_kernel(const float *__restrict__ o_part, const float *__restrict__ lse_part,
               const int *__restrict__ shard_counts, float *__restrict__ out, float *__restrict__ lse,
               int batch, int num_q_heads, int max_shards)
{
    const int lane = threadIdx.x & 31;
    const long long bh = (long long)blockIdx.x * kCombineWarps + (threadIdx.x >> 5);
    if (bh >= (long long)batch * num_q_heads) return;
    const int b = (int)(bh / num_q_heads), h = (int)(bh % num_q_heads);
    int ns = shard_counts ? shard_counts[b] : max_shards;
    ns = min(max(ns, 0), max_shards);

    const float *lrow = lse_part + ((size_t)b * max_shards) * num_q_heads + h;
    // M = max over shards of log Z; lanes stride over shards
    float M = neg_inf();
    for (int s = lane; s < ns; s += 32) M = fmaxf(M, lrow[(size_t)s * num_q_heads]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));

    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float wsum = 0.f;
    if (M != neg_inf()) {
        for (int s = 0; s < ns; ++s) {
            const float ls = lrow[(size_t)s * num_q_heads];
            if (ls == neg_inf()) continue;          // empty shard: vector never read
            const float w = expf(ls - M);           // in (0, 1]: cannot overflow
            const float4 o = *reinterpret_cast<const float4 *>(
                o_part + (((size_t)b * max_shards + s) * num_q_heads + h) * kHeadDim + lane * 4);
            wsum += w;
            acc.x = fmaf(w, o.x, acc.x);
            acc.y = fmaf(w, o.y, acc.y);
            acc.z = fmaf(w, o.z, acc.z);
            acc.w = fmaf(w, o.w, acc.w);
        }
        const float inv = 1.f / wsum;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    }
    *reinterpret_cast<float4 *>(out + (size_t)bh * kHeadDim + lane * 4) = acc;
    if (lane == 0) lse[bh] = (M == neg_inf()) ? neg_inf() : M + logf(wsum);
}

}  // namespace qf
