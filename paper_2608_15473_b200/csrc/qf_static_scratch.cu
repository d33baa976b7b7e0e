// qf_decode_partial_static: the sweep for callers that cannot allocate device memory.
//
// Some hosts of this library own no allocator they may call on the decode path: a
// serving loop whose memory pool was carved up at start-up and frozen, a plugin that
// receives only the tensors of its operator, or code running while the process is
// forbidden to call cudaMalloc (another component holds the device's allocation
// lock, or an allocation would synchronise the device in the middle of a step).
// qf_decode_partial needs a scratch buffer from its caller; this variant brings its
// own, a fixed array that lives in the library's device image.
//
// The array is a file-scope __device__ object.  In host code its name is only a
// stand-in for the symbol, not a device address, so the address is fetched once
// per device with cudaGetSymbolAddress (with that device current) and that pointer
// is what the kernels receive.
#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

#include "../../include/qf.h"

namespace {

// Every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[QF_STATIC_SCRATCH_BYTES];

std::mutex g_mu;
void *g_scratch_ptr[64];
bool g_scratch_known[64];

thread_local char g_msg[160] = "";

// The array's device address on the current device: looked up once per device, with that device current,
// after checking that the device can run this library's image at all.
int scratch_address(void **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= 64) {
        std::snprintf(g_msg, sizeof g_msg, "cudaGetDevice: %s", cudaGetErrorString(e));
        return QF_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_known[dev]) {
        int major = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) {
            std::snprintf(g_msg, sizeof g_msg, "cudaDeviceGetAttribute: %s", cudaGetErrorString(e));
            return QF_ERR_CUDA;
        }
        if (major != 10) return QF_ERR_DEVICE;   // the image holds sm_100a code only: no symbol to look up
        void *sym = nullptr;
        e = cudaGetSymbolAddress(&sym, g_static_scratch);   // the device is current: we just asked which one is
        if (e != cudaSuccess || !sym) {
            std::snprintf(g_msg, sizeof g_msg, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
            return QF_ERR_CUDA;
        }
        g_scratch_ptr[dev] = sym;
        g_scratch_known[dev] = true;
    }
    *out = g_scratch_ptr[dev];
    return QF_OK;
}

}  // namespace

extern "C" {

const char *qf_static_scratch_error(void) { return g_msg; }

int qf_decode_partial_static(const void *q, const void *k_cache, const void *v_cache,
                             const int32_t *block_table, const int32_t *seq_lens,
                             const int32_t *shard_ranges, float *o_part, float *m_part, float *lse_part,
                             const qf_params *p, void *cuda_stream)
{
    g_msg[0] = 0;
    if (!p) return QF_ERR_NULL;
    const size_t need = qf_workspace_bytes(p);
    if (need == 0) {
        // invalid parameters: nothing is looked up or set up for a call that will do nothing.  The ordinary
        // entry point names the error (its parameter check comes before it looks at the workspace).
        return qf_decode_partial(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, o_part, m_part, lse_part,
                                 p, reinterpret_cast<void *>(uintptr_t(256)), 0, cuda_stream);
    }
    if (need > (size_t)QF_STATIC_SCRATCH_BYTES) {
        std::snprintf(g_msg, sizeof g_msg,
                      "this problem needs %zu bytes of scratch but the built-in array holds %zu: "
                      "use qf_decode_partial with a caller-provided workspace",
                      need, (size_t)QF_STATIC_SCRATCH_BYTES);
        return QF_ERR_STATIC_SCRATCH;
    }
    void *ptr = nullptr;
    const int rc = scratch_address(&ptr);
    if (rc != QF_OK) return rc;
    // From here on this is exactly the ordinary sweep; its plan kernel rewrites the status
    // word and every prefix entry, and each segment state is written before it is read,
    // so nothing left over from the previous call is ever consumed.
    return qf_decode_partial(q, k_cache, v_cache, block_table, seq_lens, shard_ranges, o_part, m_part, lse_part,
                             p, ptr, (size_t)QF_STATIC_SCRATCH_BYTES, cuda_stream);
}

int qf_static_scratch_status(int32_t *host_status, void *cuda_stream)
{
    g_msg[0] = 0;
    if (!host_status) return QF_ERR_NULL;
    void *ptr = nullptr;
    const int rc = scratch_address(&ptr);
    if (rc != QF_OK) return rc;
    return qf_read_status(ptr, host_status, cuda_stream);
}

}  // extern "C"
