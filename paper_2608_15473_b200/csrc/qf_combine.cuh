// Merge of shard states (Section 5): n-way, overflow-safe form of the pairwise
// lerp / sigma / logaddexp combine.  One warp per (request, query head); each
// lane owns four channels, so a shard's 512-byte vector is one coalesced read.  A slot whose
// log Z is -inf contributes through a select, never a multiply, so garbage in it is harmless.
#pragma once

#include "qf_common.cuh"

namespace qf {

constexpr int kCombineWarps = 4;

__global__ void __launch_bounds__(kCombineWarps * 32)
combine_kernel(const float *__restrict__ o_part, const float *__restrict__ lse_part,
               const int *__restrict__ shard_counts, float *__restrict__ out, float *__restrict__ lse,
               int batch, int num_q_heads, int max_shards)
{
    grid_dependency_wait();
    grid_launch_dependents();
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
        const float *obase = o_part + (((size_t)b * max_shards) * num_q_heads + h) * kHeadDim + lane * 4;
        const size_t ostride = (size_t)num_q_heads * kHeadDim;
        for (int base = 0; base < ns; base += 32) {
            // lane s holds shard (base+s)'s weight e^{lse_s - M}: in (0, 1], cannot overflow; 0 for empty shards
            const int sl = base + lane;
            const float ls = (sl < ns) ? lrow[(size_t)sl * num_q_heads] : neg_inf();
            const float w = (ls == neg_inf()) ? 0.f : expf(ls - M);
            wsum += w;
            const int cnt = min(32, ns - base);
            for (int j = 0; j < cnt; j += 4) {
                float wj[4];
                float4 o[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {   // four independent 512-byte reads in flight
                    wj[u] = __shfl_sync(0xffffffffu, w, (j + u) & 31);
                    if (j + u >= cnt) wj[u] = 0.f;
                    o[u] = (j + u < cnt) ? *reinterpret_cast<const float4 *>(obase + (size_t)(base + j + u) * ostride)
                                         : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (wj[u] != 0.f) {         // an empty shard's vector is loaded but never used
                        acc.x = fmaf(wj[u], o[u].x, acc.x);
                        acc.y = fmaf(wj[u], o[u].y, acc.y);
                        acc.z = fmaf(wj[u], o[u].z, acc.z);
                        acc.w = fmaf(wj[u], o[u].w, acc.w);
                    }
                }
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, off);
        const float inv = 1.f / wsum;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    }
    *reinterpret_cast<float4 *>(out + (size_t)bh * kHeadDim + lane * 4) = acc;
    if (lane == 0) lse[bh] = (M == neg_inf()) ? neg_inf() : M + logf(wsum);
}

}  // namespace qf
