/*
 * qf.h -- C ABI of the Q-First cache-side decode-attention library (B200, sm_100a).
 *
 * What the library computes (Q-First paper, Section 2, on the device that needs
 * only the query, and Section 5, on splitting the cache):
 *
 *   The device that holds a request's KV cache receives the query alone, one
 *   token per request, and sweeps its cached positions.  For a set S of cached
 *   positions with scores s_i = q.k_i / sqrt(d) and values v_i,
 *       Z(S) = sum_i e^{s_i},   W(S) = sum_i e^{s_i} v_i,   O(S) = W(S)/Z(S),
 *   and the device returns (O(S), log Z(S)).  States of disjoint sets merge as
 *       O(A u B)     = lerp(O(B), O(A), sigma(log Z(A) - log Z(B))),
 *       log Z(A u B) = logaddexp(log Z(A), log Z(B)),
 *   with sigma written 1/(1+e^{-x}) so that no magnitude overflows.  An empty
 *   set is log Z = -inf and a vector that is never read.
 *
 * qf_decode_partial computes one such state per (request, KV shard, query
 * head); qf_combine merges a request's shard states into the full-context
 * attention output and its log-sum-exp.  Around them: qf_combine_self and
 * qf_append_kv (the current token's fold and cache write, Section 2),
 * qf_decode_step (sweep and merge as one call, cheaper for small sweeps),
 * qf_decode_step_host (one step from host buffers; qf_host_pipe_* the same,
 * pipelined), qf_project_pair (the
 * cache side's W_o / W_q projections at a layer boundary, Section 4),
 * qf_enable_peer_access (a request's cache split over GPUs, Section 5).
 *
 * Readings fixed at this boundary where the paper is silent:
 *   - grouped-query attention: query head h reads KV head h / G, G = Hq/Hkv;
 *   - the sweep covers cached positions [0, seq_lens[b]) only; the current
 *     token's own key/value are merged elsewhere (Section 2, the accelerator's
 *     combine) and are not part of these calls;
 *   - no causal mask, rotary embedding or normalisation inside the kernels:
 *     q and the cached keys arrive ready to be multiplied;
 *   - natural logarithm; the scale multiplies the finished fp32 dot product;
 *   - o_part is the shard-NORMALISED O(S); m_part is the running maximum
 *     score (auxiliary: W relative to m is o_part * e^{lse_part - m_part});
 *   - outputs are fp32; K, V, q are bf16.
 *
 * Memory layout (all row-major, all DEVICE memory unless stated):
 *   q            bf16  [B, Hq, D]
 *   k_cache,
 *   v_cache      bf16  [num_pages, Hkv, page_size, D]   (one (page, KV head)
 *                       block is page_size*D contiguous elements), or, with
 *                       QF_FLAG_KV_NHD, token-major pages
 *                       [num_pages, page_size, Hkv, D] (the rows of one KV
 *                       head of a page are Hkv*D elements apart).  The paper
 *                       only says that the cache is paged; both are layouts serving stacks
 *                       keep, and the results are the same bit for bit.
 *   block_table  int32 [B, max_pages_per_req]  logical page -> physical page.
 *                       May be NULL: then request b's logical page p is
 *                       physical page b*max_pages_per_req + p.
 *                       Entries past a request's last page are never read.
 *   seq_lens     int32 [B]          cached positions of each request; a length
 *                       beyond what the table row can address
 *                       (page_size * max_pages_per_req) is treated as that
 *                       limit (and reported as QF_STATUS_BAD_PAGE under
 *                       QF_FLAG_CHECK_BOUNDS): the row is never overrun
 *   shard_ranges int32 [B, S, 2]    half-open token range [beg, end) of each
 *                       shard; clamped to [0, seq_lens[b]]; beg >= end after
 *                       clamping means an empty shard.  Ranges need not be
 *                       page-aligned, balanced or disjoint.
 *   o_part       fp32  [B, S, Hq, D]
 *   m_part,
 *   lse_part     fp32  [B, S, Hq]   empty shard: -inf, and o_part = 0
 *   shard_counts int32 [B]          may be NULL (= S for every request)
 *   out          fp32  [B, Hq, D];  lse  fp32 [B, Hq]
 *
 * Ownership: every pointer is borrowed for the duration of the enqueued work;
 * the library allocates no device memory and keeps no pointer after the work
 * completes.  Its mutable state is: one-time per-device kernel attributes and
 * device properties (set under a lock); a host-side cache of TMA descriptors
 * (1,024 entries) keyed by (pointer, num_pages, num_kv_heads), also locked;
 * the fixed QF_STATIC_SCRATCH_BYTES device array that qf_decode_partial_static
 * uses, part of the library image on every GPU that loads it; and, per host
 * thread, the text of the last CUDA error, the launch count of the last call
 * and the measurement events of qf_testing.h.  `p` is host memory, read
 * before return.
 *
 * Asynchrony: every call only enqueues work on `cuda_stream` (a cudaStream_t
 * passed as void*, NULL = the legacy default stream) and returns without
 * synchronising, except qf_read_status and qf_decode_step_host, which wait.
 * qf_decode_partial and qf_combine may be captured into a CUDA graph and
 * replayed (make one un-captured call per device first: it sets kernel
 * attributes and builds the TMA descriptors); every replay tags the scratch
 * words it relies on afresh, so a replay behaves like a new call.  A workspace
 * serves one call at a time: calls that may overlap on the GPU need their own.
 *
 * Errors: 0 = success.  A negative return means nothing was enqueued.
 * Device-side metadata (table entries, ranges) is not validated unless
 * QF_FLAG_CHECK_BOUNDS is set; with it, an out-of-range page index is skipped
 * (the tokens of that page contribute nothing), recorded in the workspace
 * status word and reported by qf_read_status.  No kernel ever traps.
 */
#ifndef QF_H_
#define QF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define QF_VERSION 100

enum {
    QF_OK              = 0,
    QF_ERR_NULL        = -1, /* a required pointer is NULL                         */
    QF_ERR_BAD_SHAPE   = -2, /* non-positive size, or Hq not a multiple of Hkv     */
    QF_ERR_UNSUPPORTED = -3, /* head_dim != 128, page_size != 16, G not in 1..8     */
    QF_ERR_WORKSPACE   = -4, /* workspace NULL, misaligned (256 B) or too small    */
    QF_ERR_CUDA        = -5, /* a CUDA call failed; text via qf_strerror           */
    QF_ERR_DEVICE      = -6, /* device is not compute capability 10.x, or cannot
                                reach the peer given to qf_enable_peer_access     */
    QF_ERR_STATIC_SCRATCH = -7 /* problem too large for qf_decode_partial_static   */
};

enum {
    QF_FLAG_CHECK_BOUNDS  = 1, /* range-check page indices on the device           */
    QF_FLAG_SIMPLE_KERNEL = 2, /* use the plain-load sweep kernel (validation aid) */
    /* 8: QF_FLAG_DRAW_ALWAYS, a test hook declared in qf_testing.h                  */
    QF_FLAG_KV_NHD        = 16 /* k_cache and v_cache are [num_pages, page_size, Hkv, D]
                                  (token-major pages) instead of [num_pages, Hkv,
                                  page_size, D]; honoured by every call that touches
                                  the cache (sweep, cache write, host step)            */
};

/* qf_read_status bits */
enum {
    QF_STATUS_BAD_PAGE = 1,  /* a block-table entry was outside [0, num_pages)     */
    QF_STATUS_TIMEOUT  = 2   /* a bounded wait inside a kernel gave up             */
};

typedef struct qf_params {
    int32_t batch;             /* B                                              */
    int32_t num_q_heads;       /* Hq: a multiple of Hkv, group G = Hq/Hkv in 1..8 */
    int32_t num_kv_heads;      /* Hkv                                            */
    int32_t head_dim;          /* D, must be 128                                 */
    int32_t page_size;         /* must be 16                                     */
    int32_t max_pages_per_req; /* row stride of block_table                      */
    int32_t max_shards;        /* S: row stride of the shard arrays              */
    int32_t flags;             /* QF_FLAG_*                                      */
    int64_t num_pages;         /* pages in k_cache / v_cache                     */
    float   sm_scale;          /* <= 0 means 1/sqrt(head_dim)                    */
    int32_t out_shards;        /* qf_decode_partial only: shard slots per request of
                                  the OUTPUT arrays (0 = max_shards)             */
    int32_t out_shard_offset;  /* ... and the slot this call's shard 0 goes to    */
    int32_t max_seq_len;       /* 0, or an upper bound on seq_lens that the caller
                                  guarantees (a longer length is treated as this
                                  bound).  It lets the library recognise small
                                  sweeps when the block-table rows are much wider
                                  than the batch's contexts (see qf_decode_step)  */
} qf_params;

/* Library version (QF_VERSION of the build). */
int qf_version(void);

/* Text for a status code; for QF_ERR_CUDA includes the last CUDA error text.
 * The pointer is to static/thread-local storage owned by the library. */
const char *qf_strerror(int status);

/*
 * Bytes of device scratch qf_decode_partial needs for these parameters
 * (0 if the parameters are invalid).  The scratch holds the sweep plan
 * (prefix sums over shards), one record per piece of the schedule, segment
 * states that are merged into the per-shard states, and a status word.
 * Contents need not be initialised.
 * The pointer passed later must be 256-byte aligned.
 */
size_t qf_workspace_bytes(const qf_params *p);

/*
 * Section 2 / Section 5: the cache-side sweep.  For every request b, shard s
 * and query head h, attends q[b,h,:] over the tokens of shard s (through the
 * block table, KV head h/G) and writes the shard-normalised output, the
 * running maximum and the log-sum-exp:
 *     o_part[b,s,h,:] = O(S),  m_part[b,s,h] = max_i s_i,
 *     lse_part[b,s,h] = log Z(S).
 * Every one of the B*S slots is written (empty: 0, -inf, -inf).
 * With out_shards > 0 the outputs are laid out for a larger shard table,
 * o_part [B, out_shards, Hq, D] and m_part / lse_part [B, out_shards, Hq], and
 * this call writes slots out_shard_offset .. out_shard_offset + S - 1 of every
 * request and nothing else (Section 5: a request's cache split over devices;
 * each device sweeps the shards it holds straight into the merging device's
 * arrays, which may be peer memory: the sweep writes states with plain stores).
 * All pointers are device pointers; block_table may be NULL (identity).
 * K/V pool pointers must be 128-byte aligned.  Enqueues on cuda_stream: the
 * sweep kernel, then a small finish kernel that merges the (shard, KV head)
 * units the schedule cut into segments; a one-CTA plan kernel goes first when
 * batch * max_shards > 2,048.  The outputs are complete when the last of them
 * has run.
 */
int qf_decode_partial(const void *q, const void *k_cache, const void *v_cache,
                      const int32_t *block_table, const int32_t *seq_lens,
                      const int32_t *shard_ranges,
                      float *o_part, float *m_part, float *lse_part,
                      const qf_params *p, void *workspace, size_t workspace_bytes,
                      void *cuda_stream);

/*
 * Section 2, what the device returns for a step: the sweep of qf_decode_partial
 * and the merge of qf_combine as ONE call, same arguments, same results within
 * fp32 summation order: the shard states in o_part / m_part / lse_part and the
 * merged out [B, Hq, D], lse [B, Hq] over shards s < shard_counts[b] (NULL = all).
 * What the one call buys: a SMALL sweep is followed by one kernel instead of
 * two.  When the parameters bound the work to at most 16 stage units (of 128
 * tokens of one KV head) per SM -- batch * max_shards * num_kv_heads *
 * ceil(T / 128) <= 16 * SMs with T = min(page_size * max_pages_per_req,
 * max_seq_len), and max_shards <= 32 -- the pieces the sweep's schedule cut and
 * the request's shards are merged by a single kernel that has planned its work
 * while the sweep was still running, so that one dependent round trip to memory
 * follows the sweep instead of three to five: such a sweep is bound by launch
 * and dependent-load latency, not by bandwidth.  Larger problems enqueue the
 * same three kernels as the two calls.  out_shards must be 0 here.  Errors,
 * pointers, workspace and asynchrony as for qf_decode_partial.
 */
int qf_decode_step(const void *q, const void *k_cache, const void *v_cache,
                   const int32_t *block_table, const int32_t *seq_lens,
                   const int32_t *shard_ranges, const int32_t *shard_counts,
                   float *o_part, float *m_part, float *lse_part, float *out, float *lse,
                   const qf_params *p, void *workspace, size_t workspace_bytes,
                   void *cuda_stream);

/*
 * Section 5 across devices (a request's cache split over GPUs) with Section 3's
 * arrangement that a result is left in memory its reader can reach: before a
 * device's qf_decode_partial may store shard states into arrays that live on
 * another GPU (out_shards / out_shard_offset above, o_part / m_part / lse_part
 * being pointers into the merging GPU's memory, for example CUDA IPC mappings),
 * the CURRENT device must be allowed to access that GPU.  This call checks that
 * it can (cudaDeviceCanAccessPeer) and enables it for the calling process
 * (cudaDeviceEnablePeerAccess; already enabled counts as success; the same
 * device is a no-op).  It changes no setting of a GPU that outlasts the process.
 * Returns QF_ERR_DEVICE if the two GPUs cannot reach each other, QF_ERR_CUDA on
 * any other failure.  Only those three output arrays may be peer memory: q, the
 * KV pools, the tables and the workspace must be local to the GPU that runs the
 * call (K/V tiles are fetched by TMA, which this library never points at
 * another GPU's memory).
 */
int qf_enable_peer_access(int peer_device);

/*
 * Section 5 merge, n-way: for every (b, h), over shards s < shard_counts[b]
 * whose lse_part is not -inf,
 *     M = max_s lse_s,  w_s = e^{lse_s - M},
 *     out = sum_s w_s o_part_s / sum_s w_s,   lse = M + log sum_s w_s,
 * which is the pairwise lerp/sigma/logaddexp fold in overflow-safe form.
 * Vectors of empty shards are never read.  All shards empty: out = 0,
 * lse = -inf.  All pointers are device pointers; shard_counts may be NULL.
 */
int qf_combine(const float *o_part, const float *lse_part, const int32_t *shard_counts,
               float *out, float *lse,
               const qf_params *p, void *cuda_stream);

/*
 * Section 2, the finish of a decode step: the shard merge of qf_combine with the
 * current token folded in.  With s_jj = q.k_j/sqrt(d) for the token's own key
 * and value (k_new, v_new: bf16 [B, Hkv, D]; head h uses KV head h/G),
 *     out = lerp(v_j, o_<j, sigma(lse_<j - s_jj)),  lse = logaddexp(lse_<j, s_jj),
 * computed as one more operand (log Z = s_jj, vector v_j) of the max-subtracted
 * merge, which is the same numbers and is safe for either sign of lse_<j - s_jj
 * and for an empty cache (out = v_j, lse = s_jj).  q: bf16 [B, Hq, D].  All
 * pointers are device pointers, 8-byte aligned; shard_counts may be NULL.
 */
int qf_combine_self(const float *o_part, const float *lse_part, const int32_t *shard_counts,
                    const void *q, const void *k_new, const void *v_new,
                    float *out, float *lse,
                    const qf_params *p, void *cuda_stream);

/*
 * Section 2, the cache write (no later step of the token depends on it): stores the current token's key
 * and value (bf16 [B, Hkv, D]) at position seq_lens[b] of every request, in the
 * page block_table[b][seq_lens[b]/16] (identity table if NULL).  seq_lens is
 * not modified: the caller advances it when the next step begins.  A request
 * whose position has no allocated page (entry outside [0, num_pages), or past
 * max_pages_per_req) is skipped.  All pointers are device pointers.
 */
int qf_append_kv(void *k_cache, void *v_cache, const int32_t *block_table, const int32_t *seq_lens,
                 const void *k_new, const void *v_new,
                 const qf_params *p, void *cuda_stream);
/*
 * Section 2, the end of a decode step in ONE launch: qf_combine_self (the
 * current token folded into the swept shard states: out, lse) and qf_append_kv
 * (its key and value stored at position seq_lens[b]) together, same arguments,
 * same results bit for bit.  With advance_lengths != 0 every request whose row
 * was stored also gets seq_lens[b] += 1, after all of its KV heads have been
 * placed (a request without a page for the position keeps its length and
 * stores nothing).  The merge reads neither the cache nor the lengths, so the
 * two halves share nothing.  All pointers are device pointers; q, k_new,
 * v_new, k_cache, v_cache 8-byte aligned; shard_counts and block_table may be
 * NULL.  Errors as qf_combine_self.
 */
int qf_fold_append(const float *o_part, const float *lse_part, const int32_t *shard_counts,
                   const void *q, const void *k_new, const void *v_new,
                   float *out, float *lse,
                   void *k_cache, void *v_cache, const int32_t *block_table,
                   int32_t *seq_lens, int advance_lengths,
                   const qf_params *p, void *cuda_stream);


/*
 * Section 4 (placement: W_q and W_o live with the cache) and the appendix
 * paragraph on batching at the cache side: the projection pair at a
 * layer boundary, over the co-resident requests of a batch,
 *     u' = z + W_o a              (closes the layer:  [batch, d_model])
 *     q  = W_q N_1(u')            (opens the next:    [batch, n_q])
 * with N_1 the root-mean-square normalisation with gain g,
 *     N_1(u)_i = g_i u_i / sqrt(mean_j u_j^2 + eps).
 * The paper fixes bf16 weights and a bf16 stream; the rest is this library's
 * reading: a is the fp32 attention output (what qf_combine / qf_combine_self
 * return, [batch, n_q] = [batch, Hq, D]) and is rounded to bf16 before the
 * product; products accumulate in fp32; u' is rounded to bf16 and N_1 reads
 * the rounded stream; N_1(u') and q are rounded to bf16.  q has the layout
 * qf_decode_partial consumes.
 *   a [batch, n_q] fp32; z, u_out [batch, d_model] bf16; w_o [d_model, n_q],
 *   w_q [n_q, d_model], g [d_model] bf16, row-major; q_out [batch, n_q] bf16.
 *   All device pointers; a, z, g, u_out, q_out 16-byte aligned, the weights
 *   128-byte aligned.  workspace: qf_project_workspace_bytes bytes, 256-byte
 *   aligned, contents need not be initialised.
 * Supported: 1 <= batch <= 64; d_model and n_q multiples of 512, at most
 * 5,120; else
 * QF_ERR_UNSUPPORTED (qf_project_workspace_bytes returns 0).  Larger batches
 * are run in slices of 64 by the caller.  Enqueues two kernels on cuda_stream
 * (capturable in a CUDA graph; the first call for a shape sets kernel
 * attributes and builds the weights' TMA descriptors, so make one call
 * before capturing).  Meant for the paper's regime of a few co-resident
 * requests: from a batch of about 32 on a library GEMM is as fast or faster.
 * qf_project_status copies the pair's status word (QF_STATUS_TIMEOUT if a
 * bounded wait inside a kernel ran out; 0 = clean), clears it and synchronises
 * the stream.  The word is sticky: a bit raised by any pair that used this
 * workspace (any layer of a stack, any replay of a captured graph) stays until
 * this call has reported it once.
 */
size_t qf_project_workspace_bytes(int batch, int d_model, int n_q);
int qf_project_pair(const float *a, const void *z, const void *w_o, const void *g,
                    const void *w_q, void *u_out, void *q_out,
                    int batch, int d_model, int n_q, float eps,
                    void *workspace, size_t workspace_bytes, void *cuda_stream);
int qf_project_status(const void *workspace, int32_t *host_status, void *cuda_stream);

/*
 * One whole decode step driven from HOST buffers, as a serving loop calls it:
 * the query and the step's metadata are copied host -> device, the sweep and
 * the merge run, and the result is copied device -> host.  The KV cache stays
 * where it lives (that is the protocol: only the query travels).
 *
 *   host: q_host, seq_lens_host, shard_ranges_host, shard_counts_host (may
 *       be NULL), out_host, lse_host.  If all of them are page-locked and
 *       mapped into the device's address space (cudaHostAlloc, or
 *       cudaHostRegister with the mapped flag; out_host 16-byte aligned), no
 *       copy operation is enqueued at all: one staging kernel reads the inputs
 *       over the interconnect and the merge writes out/lse straight to the
 *       host.  Any other host memory (pageable included) takes
 *       cudaMemcpyAsync copies in and out; the results are the same bits.
 *   device: k_cache, v_cache, block_table (may be NULL), and `dev_scratch`
 *       of at least qf_step_scratch_bytes(p) bytes, 256-byte aligned, which
 *       holds the staged inputs, the shard states, the result and the sweep
 *       workspace.
 * Waits for the stream before returning, so out_host/lse_host are valid.
 */
size_t qf_step_scratch_bytes(const qf_params *p);
int qf_decode_step_host(const void *q_host, const void *k_cache, const void *v_cache,
                        const int32_t *block_table, const int32_t *seq_lens_host,
                        const int32_t *shard_ranges_host, const int32_t *shard_counts_host,
                        float *out_host, float *lse_host,
                        const qf_params *p, void *dev_scratch, size_t dev_scratch_bytes,
                        void *cuda_stream);

/*
 * The same step from host buffers, PIPELINED (Section 2: three small messages per
 * step, and only the query has to arrive before the sweep): a queue of `depth`
 * steps in flight.  qf_host_pipe_submit enqueues one step and returns at once
 * with a ticket (>= 0; negative = error code): the query and the metadata travel
 * to the device on a transfer stream of the pipe's own while earlier steps'
 * sweeps run on `cuda_stream`, the sweep and merge follow on `cuda_stream`, and
 * the result travels back on a second transfer stream while the next sweep runs.
 * qf_host_pipe_wait blocks until that ticket's out_host / lse_host are complete.
 * The caller keeps every host buffer of a step untouched from submit until its
 * wait has returned (so it rotates `depth` sets of them), and should pass
 * page-locked buffers: pageable ones make the copies synchronous.  Submitting
 * when `depth` steps are in flight first waits for the oldest.
 *   dev_scratch: qf_host_pipe_scratch_bytes(p, depth) bytes of device memory,
 *   256-byte aligned, borrowed until destroy.  depth is 1 to 8.
 * The pipe owns two CUDA streams and 3 * depth events (host-side objects; no
 * device memory is allocated).  One host thread uses a pipe at a time.
 */
typedef struct qf_host_pipe qf_host_pipe;
size_t qf_host_pipe_scratch_bytes(const qf_params *p, int depth);
int qf_host_pipe_create(qf_host_pipe **pipe, const qf_params *p, void *dev_scratch,
                        size_t dev_scratch_bytes, int depth);
long long qf_host_pipe_submit(qf_host_pipe *pipe, const void *q_host, const void *k_cache,
                              const void *v_cache, const int32_t *block_table,
                              const int32_t *seq_lens_host, const int32_t *shard_ranges_host,
                              const int32_t *shard_counts_host, float *out_host, float *lse_host,
                              void *cuda_stream);
int qf_host_pipe_wait(qf_host_pipe *pipe, long long ticket);
int qf_host_pipe_destroy(qf_host_pipe *pipe);

/*
 * Copies the workspace status word (QF_STATUS_* bits, 0 = clean) of the last
 * qf_decode_partial on this workspace to *host_status.  Synchronises the stream.
 */
int qf_read_status(const void *workspace, int32_t *host_status, void *cuda_stream);

/*
 * The sweep for callers that cannot allocate.  (The paper has no counterpart:
 * this entry point exists for the library's users, not for the method.)
 *
 * qf_decode_partial asks its caller for a scratch buffer.  Some callers have no
 * way to get one on the decode path: their device memory was partitioned at
 * start-up and the pool is closed, or they sit inside a framework operator that
 * is handed its input and output tensors and nothing else, or they run at a
 * point where calling cudaMalloc is off limits because it may block on, or
 * synchronise, the whole device.  This variant takes the same inputs and
 * outputs and no workspace: it uses a fixed array of QF_STATIC_SCRATCH_BYTES
 * that is part of the library's device image (so every GPU that loads the
 * library carries those bytes until the process ends).  It calls no cudaMalloc,
 * cudaFree or any routine that allocates.
 *
 * Limits and rules:
 *   - if qf_workspace_bytes(p) exceeds QF_STATIC_SCRATCH_BYTES the call returns
 *     QF_ERR_STATIC_SCRATCH and enqueues nothing; qf_static_scratch_error()
 *     then says how many bytes were needed.  Roughly, batch * max_shards *
 *     num_kv_heads may reach about 3,400 at a group size of 4.
 *   - the first call on each device looks the array's device address up
 *     (cudaGetSymbolAddress, with that device current) and remembers it; make
 *     that first call before starting any stream capture.
 *   - all calls on a device share the one array, which keeps whatever the last
 *     call left in it.  Each call rewrites everything it later reads (status
 *     word, plan, segment states), so back-to-back calls on one stream are
 *     safe; two calls whose kernels may overlap on the GPU (different streams,
 *     no ordering between them) race on the array and must not be issued.
 *   - qf_read_status cannot be pointed at the array from outside:
 *     qf_static_scratch_status reads the status word (QF_STATUS_* bits) of the
 *     last qf_decode_partial_static on the current device and synchronises
 *     the stream, exactly as qf_read_status does for a caller's workspace.
 * Everything else (arguments, layouts, results, error codes, asynchrony) is as
 * for qf_decode_partial.
 */
#define QF_STATIC_SCRATCH_BYTES (8u << 20)
int qf_decode_partial_static(const void *q, const void *k_cache, const void *v_cache,
                             const int32_t *block_table, const int32_t *seq_lens,
                             const int32_t *shard_ranges,
                             float *o_part, float *m_part, float *lse_part,
                             const qf_params *p, void *cuda_stream);

int qf_static_scratch_status(int32_t *host_status, void *cuda_stream);

/* Text describing the last QF_ERR_STATIC_SCRATCH / set-up failure on this thread. */
const char *qf_static_scratch_error(void);

#ifdef __cplusplus
}
#endif
#endif /* QF_H_ */
