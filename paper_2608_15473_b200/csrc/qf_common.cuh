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
    int max_tokens;          // no request is swept beyond this: min(16 * max_pages_per_req, the caller's bound)
    int max_shards;
    int out_shards;          // shard slots per request of the output arrays (>= out_shard0 + max_shards)
    int out_shard0;          // output slot of this call's shard 0
    int check_bounds;
    int draw_always;         // cut the tail into drawn chunks however short the sweep is
    int kv_nhd;              // pools are token-major [page][16][Hkv][D] instead of head-major [page][Hkv][16][D]
    long long num_pages;
    float sm_scale;
};

// Element offset of the row of (physical page, KV head c, slot t of the page) in a KV pool.
__host__ __device__ __forceinline__ size_t kv_row_offset(const DevParams &P, long long phys, int c, int t)
{
    return P.kv_nhd ? (((size_t)phys * kPageSize + t) * P.num_kv_heads + c) * kHeadDim
                    : (((size_t)phys * P.num_kv_heads + c) * kPageSize + t) * kHeadDim;
}

// Programmatic dependent launch: every kernel of the path is launched with the programmatic-stream-
// serialization attribute, so its CTAs may become resident while the previous kernel of the stream is
// still draining.  grid_dependency_wait() returns once that previous kernel has completed and its
// writes are visible: it precedes the first global read or write of every kernel.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Loads of words that other CTAs (or the previous kernel of the stream) have just written: L2-coherent
// (.cg) and pinned in program order.  The __ldcg intrinsic is a plain asm without a memory clobber, so
// the compiler may move it above a fence or a grid-dependency wait; these may not be moved.
__device__ __forceinline__ float ld_sync_f32(const float *p)
{
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long ld_sync_u64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.global.cg.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ int4 ld_sync_int4(const int4 *p)
{
    int4 v;
    asm volatile("ld.global.cg.v4.s32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000u); }

// bf16 pair packed in a 32-bit word -> two fp32 (exact).
__device__ __forceinline__ float bf16lo_to_f32(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// The workspace is never assumed to be initialised.  Words that must "start at zero" for a launch
// (the status word, the per-unit arrival counters) carry the launch's epoch in their upper 54 bits:
// a word whose epoch differs from the current launch's counts as zero.
constexpr int kEpochShift = 10;
constexpr unsigned long long kEpochLowMask = (1ull << kEpochShift) - 1;

// Header words (unsigned long long) at the start of the workspace.
enum { kHdrStatus = 0, kHdrLastEpoch = 1, kHdrTotals = 2 /* low: total units, high: units per CTA */,
       kHdrLaunchCount = 3 /* bumped by the last CTA of every sweep launch */, kHdrDone = 4 /* epoch-tagged */,
       kHdrChunk = 5 /* epoch-tagged draw counter of the unit kernel's dynamic chunks */ };

// OR `bits` into an epoch-tagged word.  Bounded retry; contention is at most a few writers.
__device__ __forceinline__ void epoch_or(unsigned long long *w, unsigned long long epoch, unsigned bits)
{
    unsigned long long old = *reinterpret_cast<volatile unsigned long long *>(w);
    for (int tries = 0; tries < (1 << 16); ++tries) {
        const unsigned long long cur = ((old >> kEpochShift) == epoch) ? (old & kEpochLowMask) : 0ull;
        const unsigned long long neu = (epoch << kEpochShift) | cur | bits;
        const unsigned long long prev = atomicCAS(w, old, neu);
        if (prev == old) return;
        old = prev;
    }
}

// Add one to an epoch-tagged counter and return the new count (0 if the bounded retry ran out).
__device__ __forceinline__ unsigned epoch_arrive(unsigned long long *w, unsigned long long epoch)
{
    unsigned long long old = *reinterpret_cast<volatile unsigned long long *>(w);
    for (int tries = 0; tries < (1 << 16); ++tries) {
        const unsigned long long cur = ((old >> kEpochShift) == epoch) ? (old & kEpochLowMask) : 0ull;
        const unsigned long long neu = (epoch << kEpochShift) | (cur + 1);
        const unsigned long long prev = atomicCAS(w, old, neu);
        if (prev == old) return (unsigned)(cur + 1);
        old = prev;
    }
    return 0;
}

// The epoch of a launch pairs the host's per-call tag (upper 30 bits) with a device-side launch count
// (lower 24 bits).  The host tag makes every API call distinct; the device count makes every REPLAY of
// a captured CUDA graph distinct (a replay re-runs the kernel with the captured host tag).  The pair is
// kept as two fields, not a sum, so that an old graph replayed after newer calls cannot land on an
// epoch a newer call used.  One thread per CTA reads the count at the CTA's start (the caller shares it
// through shared memory); the CTA that is the last to have issued all of its work (epoch-tagged done counter: by
// then every CTA of the launch has read the count) bumps it for the next launch.
__device__ __forceinline__ unsigned long long launch_epoch(const unsigned long long *header,
                                                           unsigned long long host_epoch)
{
    // an atomic read: performed at the L2 point of coherence, like the bump in launch_done
    const unsigned long long count = atomicAdd(const_cast<unsigned long long *>(header) + kHdrLaunchCount, 0ull);
    return ((host_epoch & ((1ull << 30) - 1)) << 24) | (count & ((1ull << 24) - 1));
}
// Arrival on an epoch-tagged counter that many CTAs hit at the same moment (44-bit tag, 20-bit count).
// The common case is one read and one atomicAdd (a compare-and-swap loop on the count collapses when 148
// CTAs finish together); only the first arrivals of a launch find a stale word and install a fresh one.  Returns the count
// after this arrival, or 0 if the bounded retry ran out.
__device__ __forceinline__ unsigned epoch_arrive_crowd(unsigned long long *w, unsigned long long epoch)
{
    const unsigned long long tag = epoch & ((1ull << 44) - 1);
    for (int tries = 0; tries < (1 << 12); ++tries) {
        const unsigned long long cur = *reinterpret_cast<volatile unsigned long long *>(w);
        if ((cur >> 20) == tag) {
            // fresh word: one atomicAdd, no retry loop
            const unsigned long long old = atomicAdd(w, 1ull);
            if ((old >> 20) == tag) return (unsigned)(old & 0xFFFFFull) + 1u;
        } else if (atomicCAS(w, cur, (tag << 20) | 1ull) == cur) {
            // stale word: nobody touches it except through this compare-and-swap, so exactly one
            // arrival installs the fresh word (and is its first count); the others see it next time round
            return 1u;
        }
    }
    return 0u;
}
// A counter that is drawn from with a bare atomicAdd (whose result the drawer needs only much later, so
// the round trip is off its critical path) must carry the launch's tag BEFORE the first draw.  Every CTA
// calls this once in its prologue; when it returns the word is (tag << 20 | count so far): either this
// call installed it, or another CTA's did (then the compare-and-swap fails and changes nothing).
__device__ __forceinline__ void epoch_counter_open(unsigned long long *w, unsigned long long epoch)
{
    const unsigned long long tag = epoch & ((1ull << 44) - 1);
    const unsigned long long cur = atomicAdd(w, 0ull);
    if ((cur >> 20) != tag) atomicCAS(w, cur, tag << 20);
}
__device__ __forceinline__ void launch_done(unsigned long long *header, unsigned long long epoch, unsigned n_ctas)
{
    if (epoch_arrive_crowd(header + kHdrDone, epoch) == n_ctas)
        atomicAdd(header + kHdrLaunchCount, 1ull);
}

// Row of the output arrays for entry e = b*S + s of this call: the outputs may be laid out for a larger
// shard table (a request's cache split over devices: every device writes its own slots of the merging
// device's arrays).
__device__ __forceinline__ size_t out_entry(const DevParams &P, int e)
{
    const int b = e / P.max_shards, s = e - b * P.max_shards;
    return (size_t)b * P.out_shards + P.out_shard0 + s;
}

// Clamp a shard's token range to the request's cached length, and the length to what the request's
// block-table row can address (max_tokens = 16 * max_pages_per_req): a length beyond the row is a caller
// error, and the sweep must not follow it past the row.
__device__ __forceinline__ void clamp_range(int r0, int r1, int len, int max_tokens, int &beg, int &end)
{
    beg = max(r0, 0);
    end = min(r1, min(len, max_tokens));
    if (end < beg) end = beg;
}
__host__ __device__ __forceinline__ int max_row_tokens(int max_pages_per_req) { return max_pages_per_req * kPageSize; }

// Launch with the programmatic-stream-serialization attribute (see grid_dependency_wait).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace qf
