// C ABI of the Q-First decode-attention library: argument validation, workspace
// carving and kernel launches.  See include/qf.h for the contract.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "../../include/qf.h"
#include "../../include/qf_testing.h"
#include "qf_combine.cuh"
#include "qf_common.cuh"
#include "qf_proj.cuh"
#include "qf_simple.cuh"
#include "qf_sweep.cuh"
#include "qf_merge_small.cuh"

namespace {

thread_local char g_cuda_msg[256] = "";
thread_local int g_last_launches = 0;
thread_local cudaEvent_t g_prof_start = nullptr, g_prof_stop = nullptr;

int cuda_fail(cudaError_t e, const char *what)
{
    std::snprintf(g_cuda_msg, sizeof g_cuda_msg, "%s: %s", what, cudaGetErrorString(e));
    return QF_ERR_CUDA;
}

int validate(const qf_params *p)
{
    if (!p) return QF_ERR_NULL;
    if (p->batch <= 0 || p->num_q_heads <= 0 || p->num_kv_heads <= 0 || p->max_pages_per_req <= 0 ||
        p->max_shards <= 0 || p->num_pages <= 0 || p->head_dim <= 0 || p->page_size <= 0)
        return QF_ERR_BAD_SHAPE;
    if (p->num_q_heads % p->num_kv_heads) return QF_ERR_BAD_SHAPE;
    if (p->out_shards < 0 || p->out_shard_offset < 0 || p->max_seq_len < 0) return QF_ERR_BAD_SHAPE;
    if (p->out_shards > 0 && (long long)p->out_shard_offset + p->max_shards > p->out_shards) return QF_ERR_BAD_SHAPE;
    if (p->out_shards == 0 && p->out_shard_offset != 0) return QF_ERR_BAD_SHAPE;
    if (p->head_dim != qf::kHeadDim || p->page_size != qf::kPageSize) return QF_ERR_UNSUPPORTED;
    const int G = p->num_q_heads / p->num_kv_heads;
    if (G < 1 || G > 8) return QF_ERR_UNSUPPORTED;
    // grid dimensions and 32-bit unit counts of the sweep plan
    if (p->batch > 65535 || p->num_kv_heads > 65535) return QF_ERR_UNSUPPORTED;
    if ((long long)p->batch * p->max_shards * p->num_kv_heads > (1ll << 22)) return QF_ERR_UNSUPPORTED;
    if ((long long)p->num_pages * p->num_kv_heads * qf::kPageSize >= (1ll << 31)) return QF_ERR_UNSUPPORTED;
    if ((long long)p->max_pages_per_req * qf::kPageSize >= (1ll << 31)) return QF_ERR_UNSUPPORTED;
    return QF_OK;
}

qf::DevParams dev_params(const qf_params *p)
{
    qf::DevParams d;
    d.batch = p->batch;
    d.num_q_heads = p->num_q_heads;
    d.num_kv_heads = p->num_kv_heads;
    d.group = p->num_q_heads / p->num_kv_heads;
    d.max_pages_per_req = p->max_pages_per_req;
    d.max_tokens = qf::max_row_tokens(p->max_pages_per_req);
    if (p->max_seq_len > 0 && p->max_seq_len < d.max_tokens) d.max_tokens = p->max_seq_len;
    d.max_shards = p->max_shards;
    d.out_shards = p->out_shards > 0 ? p->out_shards : p->max_shards;
    d.out_shard0 = p->out_shards > 0 ? p->out_shard_offset : 0;
    d.check_bounds = (p->flags & QF_FLAG_CHECK_BOUNDS) ? 1 : 0;
    d.draw_always = (p->flags & QF_FLAG_DRAW_ALWAYS) ? 1 : 0;
    d.kv_nhd = (p->flags & QF_FLAG_KV_NHD) ? 1 : 0;
    d.num_pages = p->num_pages;
    d.sm_scale = p->sm_scale > 0.f ? p->sm_scale : 1.0f / std::sqrt((float)p->head_dim);
    return d;
}

// One-time check per device that this is a compute-capability 10.x part (cached under a lock: any host
// thread may be the first to use a device).
int check_device(int *sm_count)
{
    static std::mutex mu;
    static int cached_major[64];
    static int cached_sms[64];
    static bool known[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return QF_ERR_DEVICE;
    std::lock_guard<std::mutex> lock(mu);
    if (!known[dev]) {
        int major = 0, sms = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
        cached_major[dev] = major;
        cached_sms[dev] = sms;
        known[dev] = true;
    }
    if (cached_major[dev] != 10) return QF_ERR_DEVICE;
    if (sm_count) *sm_count = cached_sms[dev];
    return QF_OK;
}

template <int G>
int launch_simple(const void *q, const void *k, const void *v, const int32_t *bt, const int32_t *sl,
                  const int32_t *sr, float *o, float *m, float *l, const qf::DevParams &P,
                  unsigned long long *header, unsigned long long epoch, cudaStream_t st)
{
    dim3 grid(P.max_shards, P.num_kv_heads, P.batch);
    qf::sweep_simple_kernel<G><<<grid, qf::kSimpleWarps * 32, 0, st>>>(
        (const uint16_t *)q, (const uint16_t *)k, (const uint16_t *)v, bt, sl, sr, o, m, l, P, header, epoch);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "sweep_simple_kernel launch");
    g_last_launches += 1;
    return QF_OK;
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

}  // namespace

extern "C" {

int qf_version(void) { return QF_VERSION; }

const char *qf_strerror(int status)
{
    switch (status) {
    case QF_OK: return "ok";
    case QF_ERR_NULL: return "a required pointer is NULL";
    case QF_ERR_BAD_SHAPE: return "bad shape: sizes must be positive and num_q_heads a multiple of num_kv_heads";
    case QF_ERR_UNSUPPORTED: return "unsupported: head_dim must be 128, page_size 16, group size 1 to 8";
    case QF_ERR_WORKSPACE: return "workspace is NULL, not 256-byte aligned, or too small";
    case QF_ERR_CUDA: return g_cuda_msg[0] ? g_cuda_msg : "CUDA error";
    case QF_ERR_DEVICE: return "device is not compute capability 10.x (this library is built for sm_100a only), or cannot reach the peer";
    case QF_ERR_STATIC_SCRATCH: return "problem needs more scratch than the built-in static array; use qf_decode_partial";
    default: return "unknown status";
    }
}

size_t qf_workspace_bytes(const qf_params *p)
{
    if (validate(p) != QF_OK) return 0;
    return qf::workspace_layout(p->batch, p->max_shards, p->num_kv_heads, p->num_q_heads / p->num_kv_heads).total;
}

int qf_last_launch_count(void) { return g_last_launches; }

int qf_set_profile_events(void *start_event, void *stop_event)
{
    g_prof_start = (cudaEvent_t)start_event;
    g_prof_stop = (cudaEvent_t)stop_event;
    return QF_OK;
}

namespace {
// The sweep, shared by qf_decode_partial (shard states only) and qf_decode_step (states and the merge).
// `step_out` / `step_lse` non-null: the caller wants the merged result too; *merged says whether the sweep
// kernel produced it itself (small sweeps), else the caller still has to launch the merge.
int sweep_impl(const void *q, const void *k_cache, const void *v_cache, const int32_t *block_table,
               const int32_t *seq_lens, const int32_t *shard_ranges, const int32_t *shard_counts, float *o_part,
               float *m_part, float *lse_part, float *step_out, float *step_lse, bool *merged, const qf_params *p,
               void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    g_last_launches = 0;
    if (merged) *merged = false;
    int rc = validate(p);
    if (rc != QF_OK) return rc;
    if (!q || !k_cache || !v_cache || !seq_lens || !shard_ranges || !o_part || !m_part || !lse_part)
        return QF_ERR_NULL;
    const size_t need = qf_workspace_bytes(p);
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return QF_ERR_WORKSPACE;
    if (((uintptr_t)k_cache & 127) || ((uintptr_t)v_cache & 127) || ((uintptr_t)q & 15)) return QF_ERR_BAD_SHAPE;
    int sms = 0;
    rc = check_device(&sms);
    if (rc != QF_OK) return rc;

    cudaStream_t st = (cudaStream_t)cuda_stream;
    const qf::DevParams P = dev_params(p);
    const qf::WorkspaceLayout wsl = qf::workspace_layout(P.batch, P.max_shards, P.num_kv_heads, P.group);
    unsigned long long *header = reinterpret_cast<unsigned long long *>((char *)workspace + wsl.header_off);
    const unsigned long long epoch = qf::next_epoch();

    if (p->flags & QF_FLAG_SIMPLE_KERNEL) {
        switch (P.group) {
        case 1: return launch_simple<1>(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, o_part, m_part, lse_part, P, header, epoch, st);
        case 2: return launch_simple<2>(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, o_part, m_part, lse_part, P, header, epoch, st);
        case 3: return launch_simple<3>(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, o_part, m_part, lse_part, P, header, epoch, st);
        case 4: return launch_simple<4>(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, o_part, m_part, lse_part, P, header, epoch, st);
        case 5: return launch_simple<5>(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, o_part, m_part, lse_part, P, header, epoch, st);
        case 6: return launch_simple<6>(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, o_part, m_part, lse_part, P, header, epoch, st);
        case 7: return launch_simple<7>(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, o_part, m_part, lse_part, P, header, epoch, st);
        default: return launch_simple<8>(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, o_part, m_part, lse_part, P, header, epoch, st);
        }
    }

    // A whole step over a small sweep: the sweep, then ONE kernel that merges both the pieces of cut units and
    // the request's shards (qf_merge_small.cuh) instead of the finish kernel and the merge kernel.
    const int n_ctas = sms < qf::kMaxSweepCtas ? sms : qf::kMaxSweepCtas;
    const bool small = step_out && step_lse && !(p->flags & QF_FLAG_NO_SMALL_MERGE) && p->out_shards == 0 &&
                       qf::sweep_is_small(P, n_ctas);
    int launches = 0;
    rc = qf::launch_sweep(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, o_part, m_part, lse_part, P,
                          (char *)workspace, wsl, sms, epoch, st, g_prof_start, g_prof_stop, g_cuda_msg,
                          sizeof g_cuda_msg, &launches, small);
    if (rc == QF_OK && small) {
        cudaError_t e = qf::launch_merge_small(seq_lens, shard_ranges, shard_counts, (char *)workspace, wsl, o_part,
                                               m_part, lse_part, step_out, step_lse, n_ctas, P, st);
        if (e != cudaSuccess) return cuda_fail(e, "merge_small_kernel launch");
        launches += 1;
        if (merged) *merged = true;
    }
    g_last_launches = launches;
    return rc;
}
}  // namespace

int qf_decode_partial(const void *q, const void *k_cache, const void *v_cache, const int32_t *block_table,
                      const int32_t *seq_lens, const int32_t *shard_ranges, float *o_part, float *m_part,
                      float *lse_part, const qf_params *p, void *workspace, size_t workspace_bytes,
                      void *cuda_stream)
{
    return sweep_impl(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, nullptr, o_part, m_part, lse_part,
                      nullptr, nullptr, nullptr, p, workspace, workspace_bytes, cuda_stream);
}

int qf_enable_peer_access(int peer_device)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (peer_device < 0) return QF_ERR_BAD_SHAPE;
    if (peer_device == dev) return QF_OK;
    int can = 0;
    e = cudaDeviceCanAccessPeer(&can, dev, peer_device);
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceCanAccessPeer");
    if (!can) return QF_ERR_DEVICE;
    e = cudaDeviceEnablePeerAccess(peer_device, 0);
    if (e == cudaErrorPeerAccessAlreadyEnabled) {
        cudaGetLastError();   // not an error here: clear it
        return QF_OK;
    }
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceEnablePeerAccess");
    return QF_OK;
}

namespace {
int launch_combine(const float *o_part, const float *lse_part, const int32_t *shard_counts, const void *q,
                   const void *k_new, const void *v_new, float *out, float *lse, const qf_params *p,
                   void *cuda_stream)
{
    g_last_launches = 0;
    int rc = validate(p);
    if (rc != QF_OK) return rc;
    if (!o_part || !lse_part || !out || !lse) return QF_ERR_NULL;
    rc = check_device(nullptr);
    if (rc != QF_OK) return rc;
    const qf::DevParams P = dev_params(p);
    const long long bh = (long long)p->batch * p->num_q_heads;
    const unsigned blocks = (unsigned)((bh + qf::kCombineWarps - 1) / qf::kCombineWarps);
    auto kernel = p->max_shards <= 4 ? qf::combine_kernel<4> : p->max_shards <= 8 ? qf::combine_kernel<8>
                                                                                  : qf::combine_kernel<16>;
    cudaError_t e = qf::launch_pdl(kernel, dim3(blocks), dim3(qf::kCombineWarps * 32), 0,
                                   (cudaStream_t)cuda_stream, o_part, lse_part, shard_counts, (const uint16_t *)q,
                                   (const uint16_t *)k_new, (const uint16_t *)v_new, out, lse, p->batch,
                                   p->num_q_heads, p->num_kv_heads, p->max_shards, P.sm_scale);
    if (e != cudaSuccess) return cuda_fail(e, "combine_kernel launch");
    g_last_launches = 1;
    return QF_OK;
}
}  // namespace

int qf_combine(const float *o_part, const float *lse_part, const int32_t *shard_counts, float *out, float *lse,
               const qf_params *p, void *cuda_stream)
{
    return launch_combine(o_part, lse_part, shard_counts, nullptr, nullptr, nullptr, out, lse, p, cuda_stream);
}

int qf_decode_step(const void *q, const void *k_cache, const void *v_cache, const int32_t *block_table,
                   const int32_t *seq_lens, const int32_t *shard_ranges, const int32_t *shard_counts,
                   float *o_part, float *m_part, float *lse_part, float *out, float *lse, const qf_params *p,
                   void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!out || !lse) {
        g_last_launches = 0;
        const int rc0 = validate(p);
        return rc0 != QF_OK ? rc0 : QF_ERR_NULL;
    }
    if (p && p->out_shards != 0) {   // the step owns the merge: its shard table is the whole one
        g_last_launches = 0;
        const int rc0 = validate(p);
        return rc0 != QF_OK ? rc0 : QF_ERR_BAD_SHAPE;
    }
    bool merged = false;
    int rc = sweep_impl(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, shard_counts, o_part, m_part,
                        lse_part, out, lse, &merged, p, workspace, workspace_bytes, cuda_stream);
    if (rc != QF_OK || merged) return rc;
    const int sweep_launches = g_last_launches;
    rc = qf_combine(o_part, lse_part, shard_counts, out, lse, p, cuda_stream);
    if (rc == QF_OK) g_last_launches += sweep_launches;
    return rc;
}

int qf_combine_self(const float *o_part, const float *lse_part, const int32_t *shard_counts, const void *q,
                    const void *k_new, const void *v_new, float *out, float *lse, const qf_params *p,
                    void *cuda_stream)
{
    if (!q || !k_new || !v_new) return QF_ERR_NULL;
    if (((uintptr_t)q & 7) || ((uintptr_t)k_new & 7) || ((uintptr_t)v_new & 7)) return QF_ERR_BAD_SHAPE;
    return launch_combine(o_part, lse_part, shard_counts, q, k_new, v_new, out, lse, p, cuda_stream);
}

int qf_append_kv(void *k_cache, void *v_cache, const int32_t *block_table, const int32_t *seq_lens,
                 const void *k_new, const void *v_new, const qf_params *p, void *cuda_stream)
{
    g_last_launches = 0;
    int rc = validate(p);
    if (rc != QF_OK) return rc;
    if (!k_cache || !v_cache || !seq_lens || !k_new || !v_new) return QF_ERR_NULL;
    if (((uintptr_t)k_cache & 7) || ((uintptr_t)v_cache & 7) || ((uintptr_t)k_new & 7) || ((uintptr_t)v_new & 7))
        return QF_ERR_BAD_SHAPE;
    rc = check_device(nullptr);
    if (rc != QF_OK) return rc;
    const qf::DevParams P = dev_params(p);
    const long long bc = (long long)p->batch * p->num_kv_heads;
    const unsigned blocks = (unsigned)((bc + qf::kCombineWarps - 1) / qf::kCombineWarps);
    cudaError_t e = qf::launch_pdl(qf::append_kv_kernel, dim3(blocks), dim3(qf::kCombineWarps * 32), 0,
                                   (cudaStream_t)cuda_stream, (uint16_t *)k_cache, (uint16_t *)v_cache, block_table,
                                   seq_lens, (const uint16_t *)k_new, (const uint16_t *)v_new, P);
    if (e != cudaSuccess) return cuda_fail(e, "append_kv_kernel launch");
    g_last_launches = 1;
    return QF_OK;
}

int qf_fold_append(const float *o_part, const float *lse_part, const int32_t *shard_counts, const void *q,
                   const void *k_new, const void *v_new, float *out, float *lse, void *k_cache, void *v_cache,
                   const int32_t *block_table, int32_t *seq_lens, int advance_lengths, const qf_params *p,
                   void *cuda_stream)
{
    g_last_launches = 0;
    int rc = validate(p);
    if (rc != QF_OK) return rc;
    if (!o_part || !lse_part || !out || !lse || !q || !k_new || !v_new || !k_cache || !v_cache || !seq_lens)
        return QF_ERR_NULL;
    if (((uintptr_t)q & 7) || ((uintptr_t)k_new & 7) || ((uintptr_t)v_new & 7) || ((uintptr_t)k_cache & 7) ||
        ((uintptr_t)v_cache & 7))
        return QF_ERR_BAD_SHAPE;
    rc = check_device(nullptr);
    if (rc != QF_OK) return rc;
    const qf::DevParams P = dev_params(p);
    const long long bh = (long long)p->batch * p->num_q_heads;
    const unsigned fold_blocks = (unsigned)((bh + qf::kCombineWarps - 1) / qf::kCombineWarps);
    auto kernel = p->max_shards <= 4 ? qf::fold_append_kernel<4> : p->max_shards <= 8 ? qf::fold_append_kernel<8>
                                                                                      : qf::fold_append_kernel<16>;
    cudaError_t e = qf::launch_pdl(kernel, dim3(fold_blocks + (unsigned)p->batch), dim3(qf::kCombineWarps * 32), 0,
                                   (cudaStream_t)cuda_stream, o_part, lse_part, shard_counts, (const uint16_t *)q,
                                   (const uint16_t *)k_new, (const uint16_t *)v_new, out, lse, (uint16_t *)k_cache,
                                   (uint16_t *)v_cache, block_table, (int *)seq_lens, advance_lengths != 0 ? 1 : 0,
                                   fold_blocks, P);
    if (e != cudaSuccess) return cuda_fail(e, "fold_append_kernel launch");
    g_last_launches = 1;
    return QF_OK;
}

// Carving of the step scratch used by qf_decode_step_host.
namespace {
// Device alias of a pinned, mapped host pointer; nullptr for any other kind of memory.
void *mapped_alias(const void *host)
{
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, host) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return (a.type == cudaMemoryTypeHost) ? a.devicePointer : nullptr;
}

struct StepLayout {
    size_t q, seq_lens, shard_ranges, shard_counts, o_part, m_part, lse_part, out, lse, workspace, total;
};
StepLayout step_layout(const qf_params *p)
{
    StepLayout L;
    const size_t B = p->batch, S = p->max_shards, Hq = p->num_q_heads, D = p->head_dim;
    size_t off = 0;
    L.q = off;            off = align256(off + B * Hq * D * 2);
    L.seq_lens = off;     off = align256(off + B * 4);
    L.shard_ranges = off; off = align256(off + B * S * 2 * 4);
    L.shard_counts = off; off = align256(off + B * 4);
    L.o_part = off;       off = align256(off + B * S * Hq * D * 4);
    L.m_part = off;       off = align256(off + B * S * Hq * 4);
    L.lse_part = off;     off = align256(off + B * S * Hq * 4);
    L.out = off;          off = align256(off + B * Hq * D * 4);
    L.lse = off;          off = align256(off + B * Hq * 4);
    L.workspace = off;    off = align256(off + qf_workspace_bytes(p));
    L.total = off;
    return L;
}
}  // namespace

size_t qf_step_scratch_bytes(const qf_params *p)
{
    if (validate(p) != QF_OK) return 0;
    return step_layout(p).total;
}

int qf_decode_step_host(const void *q_host, const void *k_cache, const void *v_cache, const int32_t *block_table,
                        const int32_t *seq_lens_host, const int32_t *shard_ranges_host,
                        const int32_t *shard_counts_host, float *out_host, float *lse_host, const qf_params *p,
                        void *dev_scratch, size_t dev_scratch_bytes, void *cuda_stream)
{
    int rc = validate(p);
    if (rc != QF_OK) return rc;
    if (!q_host || !k_cache || !v_cache || !seq_lens_host || !shard_ranges_host || !out_host || !lse_host)
        return QF_ERR_NULL;
    if (p->out_shards != 0) return QF_ERR_BAD_SHAPE;   // the step owns its own shard-state arrays
    const StepLayout L = step_layout(p);
    if (!dev_scratch || ((uintptr_t)dev_scratch & 255) || dev_scratch_bytes < L.total) return QF_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    char *base = (char *)dev_scratch;
    const size_t B = p->batch, S = p->max_shards, Hq = p->num_q_heads, D = p->head_dim;
    cudaError_t e;
    // Pinned, mapped host buffers are read and written by the kernels themselves: one staging launch
    // instead of four copy operations in, and the merge writes the result straight to the host, so no
    // copy operation out.  Any other kind of host memory takes the copy path.
    const void *q_dev = mapped_alias(q_host), *sl_dev = mapped_alias(seq_lens_host);
    const void *sr_dev = mapped_alias(shard_ranges_host);
    const void *sc_dev = shard_counts_host ? mapped_alias(shard_counts_host) : nullptr;
    float *out_dev = (float *)mapped_alias(out_host), *lse_dev = (float *)mapped_alias(lse_host);
    const bool mapped = q_dev && sl_dev && sr_dev && (sc_dev || !shard_counts_host) && out_dev && lse_dev &&
                        !((uintptr_t)out_dev & 15) && !((uintptr_t)q_dev & 3);
    int extra_launches = 0;
    if (mapped) {
        const qf::IngestSpan sq = {(const uint32_t *)q_dev, (uint32_t *)(base + L.q), (unsigned)(B * Hq * D / 2)};
        const qf::IngestSpan ssl = {(const uint32_t *)sl_dev, (uint32_t *)(base + L.seq_lens), (unsigned)B};
        const qf::IngestSpan ssr = {(const uint32_t *)sr_dev, (uint32_t *)(base + L.shard_ranges), (unsigned)(B * S * 2)};
        const qf::IngestSpan ssc = {(const uint32_t *)sc_dev, (uint32_t *)(base + L.shard_counts),
                                    shard_counts_host ? (unsigned)B : 0u};
        const unsigned blocks = (unsigned)std::min<size_t>(148, (B * Hq * D / 8 + 255) / 256 + 1);
        e = qf::launch_pdl(qf::ingest_kernel, dim3(blocks), dim3(256), 0, st, sq, ssl, ssr, ssc);
        if (e != cudaSuccess) return cuda_fail(e, "ingest_kernel launch");
        extra_launches = 1;
    } else {
        e = cudaMemcpyAsync(base + L.q, q_host, B * Hq * D * 2, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return cuda_fail(e, "copy q");
        e = cudaMemcpyAsync(base + L.seq_lens, seq_lens_host, B * 4, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return cuda_fail(e, "copy seq_lens");
        e = cudaMemcpyAsync(base + L.shard_ranges, shard_ranges_host, B * S * 8, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return cuda_fail(e, "copy shard_ranges");
        if (shard_counts_host) {
            e = cudaMemcpyAsync(base + L.shard_counts, shard_counts_host, B * 4, cudaMemcpyHostToDevice, st);
            if (e != cudaSuccess) return cuda_fail(e, "copy shard_counts");
        }
    }
    rc = qf_decode_step(base + L.q, k_cache, v_cache, block_table, (const int32_t *)(base + L.seq_lens),
                        (const int32_t *)(base + L.shard_ranges),
                        shard_counts_host ? (const int32_t *)(base + L.shard_counts) : nullptr,
                        (float *)(base + L.o_part), (float *)(base + L.m_part), (float *)(base + L.lse_part),
                        mapped ? out_dev : (float *)(base + L.out), mapped ? lse_dev : (float *)(base + L.lse), p,
                        base + L.workspace, dev_scratch_bytes - L.workspace, cuda_stream);
    if (rc != QF_OK) return rc;
    g_last_launches += extra_launches;
    if (!mapped) {
        e = cudaMemcpyAsync(out_host, base + L.out, B * Hq * D * 4, cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return cuda_fail(e, "copy out");
        e = cudaMemcpyAsync(lse_host, base + L.lse, B * Hq * 4, cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return cuda_fail(e, "copy lse");
    }
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    return QF_OK;
}

// ------------------------------------------------------------------------------------------------------------
// Steps from host buffers, pipelined: step n + 1's inputs travel in and step n's result travels out while a
// sweep runs.  Slots of step scratch, two private transfer streams (in, out) and three events per slot.
struct qf_host_pipe {
    qf_params p;
    char *scratch;
    size_t slot_bytes;
    int depth;
    int device;
    cudaStream_t s_in, s_out;
    cudaEvent_t ev_in[8], ev_comp[8], ev_done[8];
    long long submitted;          // tickets handed out so far
    int launches_per_step;
};

size_t qf_host_pipe_scratch_bytes(const qf_params *p, int depth)
{
    if (validate(p) != QF_OK || depth < 1 || depth > 8) return 0;
    return step_layout(p).total * (size_t)depth;
}

int qf_host_pipe_create(qf_host_pipe **pipe, const qf_params *p, void *dev_scratch, size_t dev_scratch_bytes, int depth)
{
    if (!pipe) return QF_ERR_NULL;
    *pipe = nullptr;
    int rc = validate(p);
    if (rc != QF_OK) return rc;
    if (depth < 1 || depth > 8 || p->out_shards != 0) return QF_ERR_BAD_SHAPE;
    const size_t slot = step_layout(p).total;
    if (!dev_scratch || ((uintptr_t)dev_scratch & 255) || dev_scratch_bytes < slot * (size_t)depth) return QF_ERR_WORKSPACE;
    rc = check_device(nullptr);
    if (rc != QF_OK) return rc;
    qf_host_pipe *h = new (std::nothrow) qf_host_pipe();
    if (!h) return QF_ERR_CUDA;
    h->p = *p;
    h->scratch = (char *)dev_scratch;
    h->slot_bytes = slot;
    h->depth = depth;
    h->submitted = 0;
    h->launches_per_step = 0;
    cudaGetDevice(&h->device);
    cudaError_t e = cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking);
    for (int i = 0; i < depth && e == cudaSuccess; ++i) {
        e = cudaEventCreateWithFlags(&h->ev_in[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_comp[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_done[i], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) {
        qf_host_pipe_destroy(h);   // releases whatever was created (the rest of the handles are null)
        return cuda_fail(e, "qf_host_pipe_create");
    }
    *pipe = h;
    return QF_OK;
}

long long qf_host_pipe_submit(qf_host_pipe *h, const void *q_host, const void *k_cache, const void *v_cache,
                              const int32_t *block_table, const int32_t *seq_lens_host,
                              const int32_t *shard_ranges_host, const int32_t *shard_counts_host, float *out_host,
                              float *lse_host, void *cuda_stream)
{
    if (!h || !q_host || !k_cache || !v_cache || !seq_lens_host || !shard_ranges_host || !out_host || !lse_host)
        return QF_ERR_NULL;
    const qf_params *p = &h->p;
    const long long ticket = h->submitted;
    const int slot = (int)(ticket % h->depth);
    cudaError_t e;
    if (ticket >= h->depth) {   // the slot's previous step must have left it
        e = cudaEventSynchronize(h->ev_done[slot]);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventSynchronize");
    }
    const StepLayout L = step_layout(p);
    char *base = h->scratch + (size_t)slot * h->slot_bytes;
    const size_t B = p->batch, S = p->max_shards, Hq = p->num_q_heads, D = p->head_dim;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // in: the query and the step's metadata, on the inbound stream
    e = cudaMemcpyAsync(base + L.q, q_host, B * Hq * D * 2, cudaMemcpyHostToDevice, h->s_in);
    if (e == cudaSuccess) e = cudaMemcpyAsync(base + L.seq_lens, seq_lens_host, B * 4, cudaMemcpyHostToDevice, h->s_in);
    if (e == cudaSuccess) e = cudaMemcpyAsync(base + L.shard_ranges, shard_ranges_host, B * S * 8, cudaMemcpyHostToDevice, h->s_in);
    if (e == cudaSuccess && shard_counts_host)
        e = cudaMemcpyAsync(base + L.shard_counts, shard_counts_host, B * 4, cudaMemcpyHostToDevice, h->s_in);
    if (e == cudaSuccess) e = cudaEventRecord(h->ev_in[slot], h->s_in);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, h->ev_in[slot], 0);
    if (e != cudaSuccess) return cuda_fail(e, "qf_host_pipe_submit (inbound)");
    // the step itself, on the caller's stream
    const int rc = qf_decode_step(base + L.q, k_cache, v_cache, block_table, (const int32_t *)(base + L.seq_lens),
                                  (const int32_t *)(base + L.shard_ranges),
                                  shard_counts_host ? (const int32_t *)(base + L.shard_counts) : nullptr,
                                  (float *)(base + L.o_part), (float *)(base + L.m_part), (float *)(base + L.lse_part),
                                  (float *)(base + L.out), (float *)(base + L.lse), p, base + L.workspace,
                                  h->slot_bytes - L.workspace, cuda_stream);
    if (rc != QF_OK) return rc;
    h->launches_per_step = g_last_launches;
    // out: the result, on the outbound stream
    e = cudaEventRecord(h->ev_comp[slot], st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(h->s_out, h->ev_comp[slot], 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out_host, base + L.out, B * Hq * D * 4, cudaMemcpyDeviceToHost, h->s_out);
    if (e == cudaSuccess) e = cudaMemcpyAsync(lse_host, base + L.lse, B * Hq * 4, cudaMemcpyDeviceToHost, h->s_out);
    if (e == cudaSuccess) e = cudaEventRecord(h->ev_done[slot], h->s_out);
    if (e != cudaSuccess) return cuda_fail(e, "qf_host_pipe_submit (outbound)");
    h->submitted = ticket + 1;
    return ticket;
}

int qf_host_pipe_wait(qf_host_pipe *h, long long ticket)
{
    if (!h) return QF_ERR_NULL;
    if (ticket < 0 || ticket >= h->submitted) return QF_ERR_BAD_SHAPE;
    if (ticket + h->depth < h->submitted) return QF_OK;   // its slot has been reused: that step was waited for then
    const cudaError_t e = cudaEventSynchronize(h->ev_done[(int)(ticket % h->depth)]);
    if (e != cudaSuccess) return cuda_fail(e, "cudaEventSynchronize");
    return QF_OK;
}

int qf_host_pipe_destroy(qf_host_pipe *h)
{
    if (!h) return QF_OK;
    if (h->s_in) cudaStreamSynchronize(h->s_in);
    if (h->s_out) cudaStreamSynchronize(h->s_out);
    for (int i = 0; i < h->depth; ++i) {
        if (h->ev_in[i]) cudaEventDestroy(h->ev_in[i]);
        if (h->ev_comp[i]) cudaEventDestroy(h->ev_comp[i]);
        if (h->ev_done[i]) cudaEventDestroy(h->ev_done[i]);
    }
    if (h->s_in) cudaStreamDestroy(h->s_in);
    if (h->s_out) cudaStreamDestroy(h->s_out);
    delete h;
    return QF_OK;
}

size_t qf_project_workspace_bytes(int batch, int d_model, int n_q)
{
    if (!qf::proj_shape_ok(batch, d_model, n_q) || !qf::proj_shape_ok(batch, n_q, d_model)) return 0;
    // a status word, then one row of per-request sums of squares per 128-feature tile of the stream
    return align256(256 + (size_t)(d_model / qf::kProjTileOut) * qf::kProjMaxBatch * sizeof(float));
}

int qf_project_pair(const float *a, const void *z, const void *w_o, const void *g, const void *w_q, void *u_out,
                    void *q_out, int batch, int d_model, int n_q, float eps, void *workspace, size_t workspace_bytes,
                    void *cuda_stream)
{
    g_last_launches = 0;
    if (batch < 1 || d_model < 1 || n_q < 1 || !(eps >= 0.f)) return QF_ERR_BAD_SHAPE;
    if (!qf::proj_shape_ok(batch, d_model, n_q) || !qf::proj_shape_ok(batch, n_q, d_model)) return QF_ERR_UNSUPPORTED;
    if (!a || !z || !w_o || !g || !w_q || !u_out || !q_out) return QF_ERR_NULL;
    if (((uintptr_t)a & 15) || ((uintptr_t)z & 15) || ((uintptr_t)g & 15) || ((uintptr_t)u_out & 15) ||
        ((uintptr_t)q_out & 15) || ((uintptr_t)w_o & 127) || ((uintptr_t)w_q & 127))
        return QF_ERR_BAD_SHAPE;
    const size_t need = qf_project_workspace_bytes(batch, d_model, n_q);
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return QF_ERR_WORKSPACE;
    int rc = check_device(nullptr);
    if (rc != QF_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CUtensorMap map_o, map_q;
    const int np = qf::proj_padded_batch(batch);
    const int sb_o = qf::proj_ring(n_q / (qf::kProjSplits * qf::kProjBoxK), np).sb;
    const int sb_q = qf::proj_ring(d_model / (qf::kProjSplits * qf::kProjBoxK), np).sb;
    if (qf::make_weight_map(&map_o, w_o, d_model, n_q, sb_o, g_cuda_msg, sizeof g_cuda_msg)) return QF_ERR_CUDA;
    if (qf::make_weight_map(&map_q, w_q, n_q, d_model, sb_q, g_cuda_msg, sizeof g_cuda_msg)) return QF_ERR_CUDA;
    unsigned long long *status = (unsigned long long *)workspace;
    float *ssq_part = (float *)((char *)workspace + 256);

    qf::ProjArgs s0 = {};
    s0.a = a; s0.z = (const uint16_t *)z; s0.out = (uint16_t *)u_out; s0.ssq_part = ssq_part; s0.status = status;
    s0.batch = batch; s0.n_out = d_model; s0.k_total = n_q;
    cudaError_t e = qf::launch_proj<0>(map_o, s0, st);
    if (e != cudaSuccess) return cuda_fail(e, "proj_kernel<0> launch");
    qf::ProjArgs s1 = {};
    s1.u_in = (const uint16_t *)u_out; s1.g = (const uint16_t *)g; s1.out = (uint16_t *)q_out; s1.ssq_part = ssq_part;
    s1.status = status; s1.batch = batch; s1.n_out = n_q; s1.k_total = d_model;
    s1.ssq_tiles = d_model / qf::kProjTileOut; s1.inv_d_model = 1.0f / (float)d_model; s1.eps = eps;
    e = qf::launch_proj<1>(map_q, s1, st);
    if (e != cudaSuccess) return cuda_fail(e, "proj_kernel<1> launch");
    g_last_launches = 2;
    return QF_OK;
}

int qf_project_status(const void *workspace, int32_t *host_status, void *cuda_stream)
{
    if (!workspace || !host_status) return QF_ERR_NULL;
    unsigned long long word = 0;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemcpyAsync(&word, workspace, sizeof word, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync");
    // read and clear: the bits are sticky until somebody has seen them (an untagged word reads as clean)
    e = cudaMemsetAsync(const_cast<void *>(workspace), 0, sizeof word, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    *host_status = ((word >> 8) == qf::kProjStatusTag) ? (int32_t)(word & 0xffull) : 0;
    return QF_OK;
}

namespace {
__global__ void proj_status_inject_kernel(unsigned long long *w, unsigned bits) { qf::proj_status_or(w, bits); }
}  // namespace

int qf_project_status_inject(void *workspace, int32_t bits, void *cuda_stream)
{
    if (!workspace) return QF_ERR_NULL;
    if ((uintptr_t)workspace & 255) return QF_ERR_WORKSPACE;
    int rc = check_device(nullptr);
    if (rc != QF_OK) return rc;
    proj_status_inject_kernel<<<1, 1, 0, (cudaStream_t)cuda_stream>>>((unsigned long long *)workspace,
                                                                      (unsigned)bits & 0xffu);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "proj_status_inject_kernel launch");
    return QF_OK;
}

int qf_plan_pieces(int total_units, int n_ctas, int draw_always, int32_t *piece_begin, int32_t *piece_end,
                   int capacity)
{
    if (total_units < 0 || n_ctas < 1 || n_ctas > qf::kMaxSweepCtas || capacity < 0) return QF_ERR_BAD_SHAPE;
    if (capacity > 0 && (!piece_begin || !piece_end)) return QF_ERR_NULL;
    const qf::PieceGrid g = qf::piece_grid(total_units, n_ctas, true, draw_always != 0);
    const int n = n_ctas + g.n_chunks;
    for (int p = 0; p < n && p < capacity; ++p) {
        int b, e;
        qf::piece_range(g, n_ctas, p, b, e);
        piece_begin[p] = b;
        piece_end[p] = e;
        // the inverse map the kernels use must agree with the ranges
        for (int x = b; x < e; x += (e - b > 64 ? (e - b) / 7 + 1 : 1))
            if (qf::piece_of(g, n_ctas, x) != p) return QF_ERR_BAD_SHAPE;
        if (e > b && qf::piece_of(g, n_ctas, e - 1) != p) return QF_ERR_BAD_SHAPE;
    }
    return n;
}

int qf_selftest_bounded_wait(void *workspace, void *cuda_stream)
{
    if (!workspace) return QF_ERR_NULL;
    if ((uintptr_t)workspace & 255) return QF_ERR_WORKSPACE;
    int rc = check_device(nullptr);
    if (rc != QF_OK) return rc;
    qf::selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>((unsigned long long *)workspace,
                                                                      qf::next_epoch(), 1u << 12);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "selftest_wait_kernel launch");
    return QF_OK;
}

int qf_read_status(const void *workspace, int32_t *host_status, void *cuda_stream)
{
    if (!workspace || !host_status) return QF_ERR_NULL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // word 0: status bits tagged with the epoch of the launch that set them; word 1: epoch of the last launch
    unsigned long long words[2] = {0, 0};
    cudaError_t e = cudaMemcpyAsync(words, workspace, sizeof words, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync");
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    const bool current = (words[0] >> qf::kEpochShift) == words[1];
    *host_status = current ? (int32_t)(words[0] & qf::kEpochLowMask) : 0;
    return QF_OK;
}

}  // extern "C"
