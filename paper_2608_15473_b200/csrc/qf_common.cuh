// Shared device-side definitions for the Q-First decode-attention kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace qf {

constexpr int kHeadDim  = 128;  // D
constexpr int kPageSize = 16;   // tokens per KV page
constexpr int kPageElems = kPageSize * kHeadDim;  // elements of one (page, KV head) block
constexpr int kPageBytes = kPageElems * 2;        // 4096

constexpr int kStatusBadPage = 1;
constexpr int kStatusTimeout = 2;

// Scalar launch parameters shared by every kernel.
struct DevParams {
    int batch;
    int num_q_heads;
    int num_kv_heads;
    int group;               // G = Hq / Hkv
    int max_pages_per_req;
    int max_shards;
    int check_bounds;
    long long num_pages;
    float sm_scale;
};

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000u); }

// bf16 pair packed in a 32-bit word -> two fp32 (exact).
__device__ __forceinline__ float bf16lo_to_f32(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Clamp a shard's token range to the request's cached length.
__device__ __forceinline__ void clamp_range(int r0, int r1, int len, int &beg, int &end)
{
    beg = max(r0, 0);
    end = min(r1, len);
    if (end < beg) end = beg;
}

}  // namespace qf
