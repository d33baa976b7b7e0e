// Merge of shard states (Section 5): n-way, overflow-safe form of the pairwise
// lerp / sigma / logaddexp combine.  One warp per (request, query head); each
// lane owns four channels, so a shard's 512-byte vector is one coalesced read.  A slot whose
// log Z is -inf contributes through a select, never a multiply, so garbage in it is harmless.
//
// With a current token (Section 2: s_jj = q.k_j/sqrt(d), out = lerp(v_j, o_<j, sigma(lse_<j - s_jj)),
// lse = logaddexp(lse_<j, s_jj)) the token is simply one more operand of the same merge, with
// log Z = s_jj and vector v_j: the two-way lerp/sigma form and the max-subtracted form are the
// same numbers, and the latter needs no case split on the sign of lse_<j - s_jj.
#pragma once

#include "qf_common.cuh"

namespace qf {

constexpr int kCombineWarps = 4;

// q, k_new, v_new: nullptr = no current token.  k_new, v_new: bf16 [B, Hkv, D].
// kCombineBatch: shard vectors in flight per lane (the host picks the smallest that covers max_shards,
// up to 16: fewer registers, more resident warps when shards are few).
template <int kCombineBatch>
__device__ __forceinline__ void
combine_warp(long long bh, const float *__restrict__ o_part, const float *__restrict__ lse_part,
             const int *__restrict__ shard_counts, const uint16_t *__restrict__ q,
             const uint16_t *__restrict__ k_new, const uint16_t *__restrict__ v_new,
             float *__restrict__ out, float *__restrict__ lse,
             int batch, int num_q_heads, int num_kv_heads, int max_shards, float sm_scale)
{
    const int lane = threadIdx.x & 31;
    if (bh >= (long long)batch * num_q_heads) return;
    const int b = (int)(bh / num_q_heads), h = (int)(bh % num_q_heads);
    // the current token, if any: its score against this head's query and its value row
    float s_self = neg_inf();
    float4 v_self = make_float4(0.f, 0.f, 0.f, 0.f);
    if (q != nullptr) {
        const int c = h / (num_q_heads / num_kv_heads);
        const uint2 qw = *reinterpret_cast<const uint2 *>(q + (size_t)bh * kHeadDim + lane * 4);
        const size_t row = ((size_t)b * num_kv_heads + c) * kHeadDim + lane * 4;
        const uint2 kw = *reinterpret_cast<const uint2 *>(k_new + row);
        const uint2 vw = *reinterpret_cast<const uint2 *>(v_new + row);
        float d = bf16lo_to_f32(qw.x) * bf16lo_to_f32(kw.x);
        d = fmaf(bf16hi_to_f32(qw.x), bf16hi_to_f32(kw.x), d);
        d = fmaf(bf16lo_to_f32(qw.y), bf16lo_to_f32(kw.y), d);
        d = fmaf(bf16hi_to_f32(qw.y), bf16hi_to_f32(kw.y), d);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
        s_self = d * sm_scale;
        v_self = make_float4(bf16lo_to_f32(vw.x), bf16hi_to_f32(vw.x), bf16lo_to_f32(vw.y), bf16hi_to_f32(vw.y));
    }

    // Everything the merge reads is requested before anything is waited for: the shard count, the first 32
    // log Z values (lane s holds shard s) and the first kCombineBatch shard vectors go out together, one
    // round trip to L2 for the usual shard counts.  Slots at or beyond the shard count exist (the arrays
    // have max_shards slots per request) but may hold anything: they are masked below, never multiplied.
    const float *lrow = lse_part + ((size_t)b * max_shards) * num_q_heads + h;
    const float *obase = o_part + (((size_t)b * max_shards) * num_q_heads + h) * kHeadDim + lane * 4;
    const size_t ostride = (size_t)num_q_heads * kHeadDim;
    const float ls_first = (lane < max_shards) ? lrow[(size_t)lane * num_q_heads] : neg_inf();
    float4 o[kCombineBatch];
#pragma unroll
    for (int u = 0; u < kCombineBatch; ++u)
        o[u] = (u < max_shards) ? *reinterpret_cast<const float4 *>(obase + (size_t)u * ostride)
                                : make_float4(0.f, 0.f, 0.f, 0.f);
    bool loaded = true;   // o[] holds shards 0 .. kCombineBatch-1
    int ns = shard_counts ? shard_counts[b] : max_shards;
    ns = min(max(ns, 0), max_shards);

    // M = max over operands of log Z; lanes stride over shards
    float M = s_self;
    if (lane < ns) M = fmaxf(M, ls_first);
    for (int s = lane + 32; s < ns; s += 32) M = fmaxf(M, lrow[(size_t)s * num_q_heads]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));

    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float wsum = 0.f;
    if (M != neg_inf()) {
        for (int base = 0; base < ns; base += 32) {
            // lane s holds shard (base+s)'s weight e^{lse_s - M}: in (0, 1], cannot overflow; 0 for empty shards
            const int sl = base + lane;
            float ls = neg_inf();
            if (sl < ns) ls = (base == 0) ? ls_first : lrow[(size_t)sl * num_q_heads];
            const float w = (ls == neg_inf()) ? 0.f : expf(ls - M);
            wsum += w;
            const int cnt = min(32, ns - base);
            for (int j = 0; j < cnt; j += kCombineBatch) {
                if (!loaded) {
#pragma unroll
                    for (int u = 0; u < kCombineBatch; ++u)   // independent 512-byte reads in flight together
                        o[u] = (j + u < cnt) ? *reinterpret_cast<const float4 *>(obase + (size_t)(base + j + u) * ostride)
                                             : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                loaded = false;
#pragma unroll
                for (int u = 0; u < kCombineBatch; ++u) {
                    const float wu = __shfl_sync(0xffffffffu, w, (j + u) & 31);
                    if (j + u < cnt && wu != 0.f) {   // an empty shard's vector is loaded but never used
                        acc.x = fmaf(wu, o[u].x, acc.x);
                        acc.y = fmaf(wu, o[u].y, acc.y);
                        acc.z = fmaf(wu, o[u].z, acc.z);
                        acc.w = fmaf(wu, o[u].w, acc.w);
                    }
                }
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, off);
        if (s_self != neg_inf()) {
            const float w = expf(s_self - M);
            wsum += w;
            acc.x = fmaf(w, v_self.x, acc.x);
            acc.y = fmaf(w, v_self.y, acc.y);
            acc.z = fmaf(w, v_self.z, acc.z);
            acc.w = fmaf(w, v_self.w, acc.w);
        }
        const float inv = 1.f / wsum;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    }
    *reinterpret_cast<float4 *>(out + (size_t)bh * kHeadDim + lane * 4) = acc;
    if (lane == 0) lse[bh] = (M == neg_inf()) ? neg_inf() : M + logf(wsum);
}

template <int kCombineBatch>
__global__ void __launch_bounds__(kCombineWarps * 32)
combine_kernel(const float *__restrict__ o_part, const float *__restrict__ lse_part,
               const int *__restrict__ shard_counts, const uint16_t *__restrict__ q,
               const uint16_t *__restrict__ k_new, const uint16_t *__restrict__ v_new,
               float *__restrict__ out, float *__restrict__ lse,
               int batch, int num_q_heads, int num_kv_heads, int max_shards, float sm_scale)
{
    grid_dependency_wait();
    grid_launch_dependents();
    combine_warp<kCombineBatch>((long long)blockIdx.x * kCombineWarps + (threadIdx.x >> 5), o_part, lse_part,
                                shard_counts, q, k_new, v_new, out, lse, batch, num_q_heads, num_kv_heads, max_shards,
                                sm_scale);
}

// The cache write of Section 2 (no later step of the token depends on it): the current token's key and value go to position
// seq_lens[b] of request b, through the block table.  One warp per (request, KV head).
// Physical page of position pos of request b, or -1 if the request has no page for it.
__device__ __forceinline__ long long append_page(const int *__restrict__ block_table, int b, int pos, const DevParams &P)
{
    const int lp = pos >> 4;
    if (pos < 0 || lp >= P.max_pages_per_req) return -1;
    const long long phys = block_table ? (long long)block_table[(size_t)b * P.max_pages_per_req + lp]
                                       : (long long)b * P.max_pages_per_req + lp;
    return (phys < 0 || phys >= P.num_pages) ? -1 : phys;
}
// One warp writes the rows of (request b, KV head c) at position pos of physical page phys.
__device__ __forceinline__ void append_row(uint16_t *__restrict__ k_cache, uint16_t *__restrict__ v_cache,
                                           const uint16_t *__restrict__ k_new, const uint16_t *__restrict__ v_new,
                                           int b, int c, int pos, long long phys, const DevParams &P)
{
    const int lane = threadIdx.x & 31;
    const size_t dst = kv_row_offset(P, phys, c, pos & 15) + lane * 4;
    const size_t src = ((size_t)b * P.num_kv_heads + c) * kHeadDim + lane * 4;
    *reinterpret_cast<uint2 *>(k_cache + dst) = *reinterpret_cast<const uint2 *>(k_new + src);
    *reinterpret_cast<uint2 *>(v_cache + dst) = *reinterpret_cast<const uint2 *>(v_new + src);
}
__global__ void __launch_bounds__(kCombineWarps * 32)
append_kv_kernel(uint16_t *__restrict__ k_cache, uint16_t *__restrict__ v_cache,
                 const int *__restrict__ block_table, const int *__restrict__ seq_lens,
                 const uint16_t *__restrict__ k_new, const uint16_t *__restrict__ v_new, DevParams P)
{
    grid_dependency_wait();
    grid_launch_dependents();
    const long long bc = (long long)blockIdx.x * kCombineWarps + (threadIdx.x >> 5);
    if (bc >= (long long)P.batch * P.num_kv_heads) return;
    const int b = (int)(bc / P.num_kv_heads), c = (int)(bc % P.num_kv_heads);
    const int pos = seq_lens[b];
    const long long phys = append_page(block_table, b, pos, P);
    if (phys < 0) return;   // no page for this position, or an unallocated one: nothing is written
    append_row(k_cache, v_cache, k_new, v_new, b, c, pos, phys, P);
}

// The end of a decode step in one launch (Section 2): the first fold_blocks CTAs fold the current token into the
// swept shard states (the merge above), the others, one per request, write the token's key and value into the cache
// at position seq_lens[b] and, if asked, advance that length — after every row of the request has been placed, and
// only if the position had a page.  The merge reads neither the cache nor the lengths, so the two halves share nothing.
template <int kCombineBatch>
__global__ void __launch_bounds__(kCombineWarps * 32)
fold_append_kernel(const float *__restrict__ o_part, const float *__restrict__ lse_part,
                   const int *__restrict__ shard_counts, const uint16_t *__restrict__ q,
                   const uint16_t *__restrict__ k_new, const uint16_t *__restrict__ v_new,
                   float *__restrict__ out, float *__restrict__ lse, uint16_t *__restrict__ k_cache,
                   uint16_t *__restrict__ v_cache, const int *__restrict__ block_table, int *__restrict__ seq_lens,
                   int advance, unsigned fold_blocks, DevParams P)
{
    grid_dependency_wait();
    grid_launch_dependents();
    if (blockIdx.x < fold_blocks) {
        combine_warp<kCombineBatch>((long long)blockIdx.x * kCombineWarps + (threadIdx.x >> 5), o_part, lse_part,
                                    shard_counts, q, k_new, v_new, out, lse, P.batch, P.num_q_heads, P.num_kv_heads,
                                    P.max_shards, P.sm_scale);
        return;
    }
    const int b = (int)(blockIdx.x - fold_blocks);
    const int pos = seq_lens[b];
    const long long phys = append_page(block_table, b, pos, P);
    if (phys < 0) return;                       // the same for every thread of the CTA
    for (int c = threadIdx.x >> 5; c < P.num_kv_heads; c += kCombineWarps)
        append_row(k_cache, v_cache, k_new, v_new, b, c, pos, phys, P);
    __syncthreads();                            // every warp has read the length and placed its rows
    if (advance && threadIdx.x == 0) seq_lens[b] = pos + 1;
}

// Staging of a decode step's inputs from pinned, mapped host memory: the kernel reads the host buffers
// over the interconnect itself (four spans, one launch) instead of four copy-engine operations.
// Spans are sequences of 32-bit words; `words16` of them, from the start, move as 16-byte words.
struct IngestSpan {
    const uint32_t *src;   // device alias of the host buffer
    uint32_t *dst;
    unsigned words;        // 32-bit words
};
__global__ void __launch_bounds__(256)
ingest_kernel(IngestSpan a, IngestSpan b, IngestSpan c, IngestSpan d)
{
    grid_dependency_wait();
    grid_launch_dependents();
    const unsigned tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
    const IngestSpan spans[4] = {a, b, c, d};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const IngestSpan sp = spans[k];
        if (sp.words == 0) continue;
        const bool wide = (((uintptr_t)sp.src | (uintptr_t)sp.dst) & 15) == 0;
        const unsigned n16 = wide ? sp.words / 4 : 0;
        for (unsigned i = tid; i < n16; i += nth)
            reinterpret_cast<uint4 *>(sp.dst)[i] = reinterpret_cast<const uint4 *>(sp.src)[i];
        for (unsigned i = n16 * 4 + tid; i < sp.words; i += nth) sp.dst[i] = sp.src[i];
    }
}

}  // namespace qf
