/*
 * ls.h -- C ABI of the B200 (sm_100a) exact-attention response-replay library.
 *
 * The library computes the hot path of LongStraw's GRPO transaction
 * (arxiv 2607.14952): one response suffix of R tokens attends causally to a long,
 * resident, gradient-free prefix of P positions whose K/V live on explicitly
 * owned physical pages.  The prefix is cut into S shards (the paper's
 * context-parallel ranks, here all on one GPU); every shard yields a normalised
 * partial output and its row log-normaliser (Eq. qwen-local-attn), the partials
 * are composed by the stable LSE/output merge (Eq. qwen-lse-parts,
 * Eq. qwen-global-attn), and the backward returns dQ (the sum of per-shard
 * contributions, Eq. qwen-dq-reduce) plus dK/dV of the response tokens only --
 * prefix pages never receive a gradient (Sec. "Lazy Gradient Pages").
 *
 * Conventions
 *  - Every tensor pointer is a DEVICE pointer unless its comment says "host".
 *  - bf16 tensors are dense in their last dimension; Q/K_resp/V_resp/dO and all
 *    outputs are fully contiguous in the stated shape.  All bases 16-byte aligned.
 *  - The caller owns every buffer, including the page pool and the workspaces.
 *    The library owns only the opaque ls_pages_t handle and its small metadata
 *    arrays, and never writes the pool.
 *  - All compute calls enqueue work on `stream` (a cudaStream_t passed as
 *    void*, NULL = default stream) and return without synchronising.  They
 *    allocate nothing.
 *  - Every call returns an ls_status_t; nothing aborts or throws across the ABI.
 *    Argument, shape, alignment and page-table validation happen on the host
 *    before any launch.  Conditions found on the device (a bounded wait that ran
 *    out) are written to `status_dev` (one int32, nullable, must be zeroed by
 *    the caller) and never trap.
 *  - GQA: query head h uses KV head h / (num_q_heads / num_kv_heads).
 *  - Response query t sits at global position P + t; it sees every prefix
 *    position and the response positions j <= t.
 *  - Results are deterministic: no floating-point atomics anywhere.
 *
 * Supported shapes: (dim_k, dim_v) in {(128,128), (256,256), (576,512)},
 * page_size in {64,128,256,512}, num_q_heads % num_kv_heads == 0.
 */
#ifndef LS_H_
#define LS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ls_pages ls_pages_t;   /* opaque handle: page table + shard plan */

typedef enum {
  LS_OK = 0,
  LS_ERR_INVALID_ARG = -1,
  LS_ERR_BAD_PAGE_TABLE = -2,
  LS_ERR_UNSUPPORTED_SHAPE = -3,
  LS_ERR_ALIGNMENT = -4,
  LS_ERR_WORKSPACE = -5,
  LS_ERR_STALE = -6,
  LS_ERR_CUDA = -7,
  LS_ERR_TIMEOUT = -8,
  LS_ERR_NONFINITE = -9
} ls_status_t;

typedef enum {
  LS_SHARD_CONTIGUOUS = 0,  /* shard s = one contiguous run of logical pages; when S does not
                               divide Np the first Np mod S shards hold one page more */
  LS_SHARD_CYCLIC = 1,      /* Eq. qwen-page-owner: owner(p) = p mod S */
  LS_SHARD_ZIGZAG = 2       /* Eq. glm-tr-zigzag-pages: shard r owns chunk r then chunk 2S-1-r of
                               2S contiguous chunks (same uneven-split rule over 2S chunks) */
} ls_shard_policy_t;

/* Describes the caller-owned physical page pool.  Strides are in ELEMENTS (bf16). */
typedef struct {
  int64_t prefix_len;      /* P >= 0 */
  int32_t page_size;       /* tokens per page */
  int32_t num_shards;      /* S >= 1 */
  int32_t shard_policy;    /* ls_shard_policy_t */
  int32_t num_kv_heads;
  int32_t dim_k;
  int32_t dim_v;
  int32_t v_aliases_k;     /* 1: V is the first dim_v channels of the K page (shared latent);
                              v_pool may then be NULL */
  int32_t reserved;
  int64_t num_phys_pages;  /* pool capacity, >= ceil(P / page_size) */
  const void* k_pool;      /* [num_phys_pages, page_size, num_kv_heads, dim_k] bf16, or NULL */
  const void* v_pool;      /* [num_phys_pages, page_size, num_kv_heads, dim_v] bf16, or NULL */
  int64_t k_stride_page, k_stride_tok, k_stride_head;
  int64_t v_stride_page, v_stride_tok, v_stride_head;
} ls_pages_desc_t;

/*
 * Page table plus shard boundaries (Sec. "From Logical Shards to Physical Pages").
 * phys_of_logical: host array of ceil(P/page_size) physical page ids, one-to-one into
 * [0, num_phys_pages); NULL means the identity.  The last logical page holds
 * P - (Np-1)*page_size valid tokens.  With k_pool == NULL the handle is a host-only
 * plan (export works, attention calls return LS_ERR_INVALID_ARG) and no CUDA call is
 * made; otherwise the plan is uploaded to the current device (small cudaMalloc) and
 * the pool's TMA descriptors are encoded.  On error *out is NULL.
 * Errors: LS_ERR_INVALID_ARG, LS_ERR_UNSUPPORTED_SHAPE, LS_ERR_BAD_PAGE_TABLE
 * (range / duplicate), LS_ERR_ALIGNMENT, LS_ERR_CUDA.
 */
ls_status_t ls_prefix_pages_build(const ls_pages_desc_t* desc, const int32_t* phys_of_logical,
                                  ls_pages_t** out);

/*
 * Copies the plan to host arrays (any may be NULL):
 *  page_table[Np]        physical id of logical page p
 *  shard_of_page[Np]     owner shard of logical page p
 *  shard_page_offset[S+1] prefix sums of pages per shard
 *  shard_logical_pages[Np] logical pages of shard 0, then shard 1, ... in local order
 *  shard_tokens[S]       valid tokens per shard
 */
ls_status_t ls_prefix_pages_export(const ls_pages_t* pages, int32_t* page_table, int32_t* shard_of_page,
                                   int64_t* shard_page_offset, int32_t* shard_logical_pages,
                                   int64_t* shard_tokens);

/*
 * 64-bit checksum over the bytes of every mapped K (and V) page, in logical order
 * (Sec. "Multi-step resident prefix reuse": the prefix must be unmodified between
 * replays).  scratch_dev: one uint64 on the device.  Synchronises `stream` and writes
 * the result to the host word *out.  Integer arithmetic only: equal bytes give equal sums.
 */
ls_status_t ls_prefix_pages_checksum(const ls_pages_t* pages, uint64_t* scratch_dev, uint64_t* out,
                                     void* stream);

ls_status_t ls_prefix_pages_destroy(ls_pages_t* pages);

typedef struct {
  int32_t R;             /* response tokens, >= 1 */
  int32_t num_q_heads;   /* Hq */
  float scale;           /* softmax scale, e.g. 1/sqrt(dim_k) */
  int32_t flags;         /* 0, or LS_FLAG_* bits */
} ls_attn_params_t;

/* Diagnostic switches for profiling the kernel pipelines: they skip one stage (operand
 * loads, tensor-core instructions, or the per-row arithmetic) while keeping every barrier
 * hand-off, so the cost of the remaining stages can be timed.  Outputs are meaningless
 * when any of them is set. */
#define LS_FLAG_ABLATE_LOADS   (1 << 16)
#define LS_FLAG_ABLATE_MMA     (1 << 17)
#define LS_FLAG_ABLATE_SOFTMAX (1 << 18)
#define LS_FLAG_ABLATE_MASK    (7 << 16)

enum { LS_WORKSPACE_FWD = 0, LS_WORKSPACE_BWD = 1 };

/* Bytes of caller-provided scratch needed by the forward (0) or the backward. */
size_t ls_replay_attn_workspace_bytes(const ls_pages_t* pages, const ls_attn_params_t* prm, int which);

/*
 * Per-shard replay forward (Eq. qwen-local-attn) plus the causal response block as
 * partial index S:
 *   lse_part[r,t,h] = log sum_{j in K_r} exp(scale q_th . k_j)      (natural log)
 *   o_part[r,t,h,:] = sum_{j in K_r} exp(s_tj - lse_part) v_j
 * An empty partial has lse = -inf and o = 0.
 *  q [R,Hq,dim_k] bf16; k_resp [R,Hkv,dim_k], v_resp [R,Hkv,dim_v] bf16
 *  o_part [(S+1),R,Hq,dim_v] fp32; lse_part [(S+1),R,Hq] fp32
 *  workspace: ls_replay_attn_workspace_bytes(.., LS_WORKSPACE_FWD) bytes of device memory,
 *  16-byte aligned; 0 (workspace may be NULL) unless the plan splits a shard into
 *  cache-sized sub-shards, whose partials are held there and merged per shard with the same
 *  Eq. qwen-lse-parts arithmetic before the call returns its (S+1) partials.  A workspace
 *  that is too small gives LS_ERR_WORKSPACE before any launch.
 */
ls_status_t ls_replay_attn_fwd(const ls_pages_t* pages, const ls_attn_params_t* prm,
                               const void* q, const void* k_resp, const void* v_resp,
                               float* o_part, float* lse_part,
                               void* workspace, size_t workspace_bytes,
                               int32_t* status_dev, void* stream);

/*
 * Stable LSE/output merge (Eq. qwen-lse-parts, Eq. qwen-global-attn) over num_parts
 * partials of `rows` rows:  m = max_r l_r; a = sum_r e^{l_r-m}; n = sum_r e^{l_r-m} o_r;
 * o = n/a; l = m + log a.  fp32 throughout; a partial with l_r = -inf weighs exactly 0.
 *  o_part [num_parts, rows, dim_v] fp32; lse_part [num_parts, rows] fp32
 *  o_bf16 [rows, dim_v] bf16 (nullable); o_f32 [rows, dim_v] fp32 (nullable; the backward
 *  consumes it); lse [rows] fp32.
 */
ls_status_t ls_lse_merge(int32_t num_parts, int64_t rows, int32_t dim_v,
                         const float* o_part, const float* lse_part,
                         void* o_bf16, float* o_f32, float* lse, void* stream);

/*
 * Replay backward with the prefix detached (Sec. "Lazy Gradient Pages"):
 *   Delta = dO.O; p_tj = exp(s_tj - LSE); ds_tj = p_tj (dO_th.v_j - Delta)
 *   dQ_th = scale * sum_j ds_tj k_j over prefix and response keys; per-shard
 *           contributions are summed on the device (Eq. qwen-dq-reduce)
 *   dK_resp_j = scale * sum_{t>=j,h in group} ds_tj q_th;  dV_resp_j = sum p_tj dO_th
 * Prefix pages get no gradient and are not written.
 *  o_f32 [R,Hq,dim_v], lse [R,Hq] from ls_lse_merge; d_o [R,Hq,dim_v] bf16
 *  dq [R,Hq,dim_k], dk_resp [R,Hkv,dim_k], dv_resp [R,Hkv,dim_v] bf16
 */
ls_status_t ls_replay_attn_bwd(const ls_pages_t* pages, const ls_attn_params_t* prm,
                               const void* q, const void* k_resp, const void* v_resp,
                               const float* o_f32, const float* lse, const void* d_o,
                               void* dq, void* dk_resp, void* dv_resp,
                               void* workspace, size_t workspace_bytes,
                               int32_t* status_dev, void* stream);

/*
 * ls_replay_attn_bwd for callers that cannot hand over scratch memory (the paper has no
 * counterpart; this is a packaging variant, the arithmetic and the outputs are those of
 * ls_replay_attn_bwd).  A replay scheduler that has sized the page pool to fill the GPU, or
 * code running under a framework whose allocator already owns all device memory, has
 * nowhere to take a workspace from at backward time: a late cudaMalloc there can fail or
 * stall the whole device.  This call therefore allocates nothing, in the library or in
 * CUDA: the per-partial dQ sums and Delta go to a fixed array of LS_STATIC_SCRATCH_BYTES
 * that is part of the library's device image, so every GPU that loads the library holds
 * that much memory until the process exits.
 *  - Shapes whose backward workspace (ls_replay_attn_workspace_bytes) exceeds
 *    LS_STATIC_SCRATCH_BYTES are rejected with LS_ERR_WORKSPACE before any launch.
 *  - The first call on each device looks up the array's device address (the device must be
 *    current); make that first call before starting any stream capture.
 *  - All calls on a device share the one array, which keeps the previous call's contents.
 *    Nothing needs clearing (every word that is read is written first by the same call),
 *    but two calls whose kernels overlap on the GPU (different streams) race on it:
 *    serialise them.
 * Arguments and errors otherwise as ls_replay_attn_bwd.
 */
#define LS_STATIC_SCRATCH_BYTES (32u << 20)
size_t ls_replay_attn_bwd_static_capacity(void);
ls_status_t ls_replay_attn_bwd_static(const ls_pages_t* pages, const ls_attn_params_t* prm,
                                      const void* q, const void* k_resp, const void* v_resp,
                                      const float* o_f32, const float* lse, const void* d_o,
                                      void* dq, void* dk_resp, void* dv_resp,
                                      int32_t* status_dev, void* stream);

/*
 * Measurement aid (the paper has no counterpart): arms a one-shot pair of CUDA events
 * (cudaEvent_t passed as void*) that the NEXT launch of the named kernel records on its
 * own stream, start just before and stop just after the launch.  The pair is disarmed
 * once used.  Passing NULL events disarms.  Not thread-safe; meant for benchmarks.
 */
typedef enum {
  LS_KERNEL_FWD = 0,      /* replay forward (one launch per ls_replay_attn_fwd) */
  LS_KERNEL_BWD_DQ = 1,   /* query-gradient pass over all partials */
  LS_KERNEL_BWD_DK = 2,   /* response dK pass */
  LS_KERNEL_BWD_DV = 3,   /* response dV pass */
  LS_KERNEL_COUNT = 4
} ls_kernel_t;
ls_status_t ls_profile_arm_events(int kernel, void* start_event, void* stop_event);

/*
 * Self-test of the bounded device-side wait (the paper has no counterpart).  Launches one
 * small CTA whose thread waits, with the library's own wait routine and a budget of
 * `budget_ns` nanoseconds, on a barrier that nothing ever completes.  The wait must give up,
 * the kernel must exit normally and LS_ERR_TIMEOUT must appear in *status_dev (device int32,
 * zeroed by the caller).  Nothing traps, faults or spins without bound.
 */
ls_status_t ls_selftest_bounded_wait(int32_t* status_dev, uint64_t budget_ns, void* stream);

const char* ls_status_string(ls_status_t status);

#ifdef __cplusplus
}
#endif
#endif  /* LS_H_ */
