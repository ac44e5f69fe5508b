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
 *    arrays.  It never writes a pool page that the prefix maps; the only pool pages
 *    it writes are the unmapped ones a caller hands to ls_suffix_pages_append.
 *  - All compute calls enqueue work on `stream` (a cudaStream_t passed as
 *    void*, NULL = default stream) and return without synchronising.  They
 *    allocate nothing.
 *  - Every call returns an ls_status_t; nothing aborts or throws across the ABI.
 *    Argument, shape, alignment and page-table validation happen on the host
 *    before any launch.  Conditions found on the device (a bounded wait that ran
 *    out, a non-finite merged log-normaliser) are written to `status_dev` (one
 *    int32, nullable, must be zeroed by the caller) and never trap.
 *  - A handle belongs to the device that was current in ls_prefix_pages_build; a
 *    compute call made with another device current returns LS_ERR_STALE.
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
  LS_ERR_STALE = -6,       /* handle of another device, or its suffix changed since the caller looked */
  LS_ERR_CUDA = -7,
  LS_ERR_TIMEOUT = -8,     /* device side: a bounded wait ran out */
  LS_ERR_NONFINITE = -9    /* device side: a merged log-normaliser is NaN or +inf */
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
  int32_t stream_budget_kib; /* 0 = default (32768).  Upper bound, in KiB, for the K+V bytes of one
                              (KV head, key range) stream that many CTAs read together: a shard above
                              it is walked as up to 16 consecutive sub-ranges, which keeps the stream
                              in L2.  Results do not depend on it beyond fp32 summation order. */
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
 * plan (export works, attention calls return LS_ERR_INVALID_ARG -- also for P = 0: a
 * handle used for attention needs a pool of at least one page) and no CUDA call is
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
  int32_t R;             /* response tokens of this call (a whole response, or one block of it), >= 1 */
  int32_t num_q_heads;   /* Hq */
  float scale;           /* softmax scale, e.g. 1/sqrt(dim_k) */
  int32_t flags;         /* 0, or LS_FLAG_* bits */
  uint64_t generation;   /* 0 = not checked; otherwise the value of ls_pages_generation() the caller
                            planned this call against: a handle whose suffix changed since then
                            (append / pop) makes the call return LS_ERR_STALE before any launch */
} ls_attn_params_t;

/* Backward only: add the retained suffix gradient pages of the block that was popped last
 * (the one being replayed) to dk_resp / dv_resp.  See ls_suffix_pages_append. */
#define LS_FLAG_ADD_SUFFIX_GRAD (1 << 0)
/* Forward and backward: leave the causal response block out.  The call then covers the prefix
 * (and suffix) parts only: k_resp / v_resp / dk_resp / dv_resp are not used (may be NULL), the
 * forward writes the response block's partial as empty, dQ sums the remaining parts.  Used to
 * compose attention over several key sets that share one response (sparse replay). */
#define LS_FLAG_NO_RESPONSE_BLOCK (1 << 1)

enum { LS_WORKSPACE_FWD = 0, LS_WORKSPACE_BWD = 1, LS_WORKSPACE_FWD_MERGED = 2 };

/* Bytes of caller-provided scratch needed by ls_replay_attn_fwd (0), ls_replay_attn_bwd (1) or
 * ls_replay_attn_fwd_merged (2).  Depends on the handle and on prm->R, prm->num_q_heads only. */
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
 *  16-byte aligned: 0 (workspace may be NULL) unless a shard is walked as several
 *  sub-ranges (stream_budget_kib), in which case it holds a few KB of hand-over counters:
 *  the CTAs of consecutive sub-ranges fold their results into the shard's partial in a
 *  fixed order with the Eq. qwen-lse-parts arithmetic, so the caller still receives (S+1)
 *  partials and no per-sub-range partial ever exists in memory.  A workspace that is too
 *  small gives LS_ERR_WORKSPACE before any launch.
 * The handle must have no suffix blocks (LS_ERR_INVALID_ARG): use ls_replay_attn_fwd_merged.
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
 * A merged l that is NaN or +inf (only possible from non-finite inputs) is still written,
 * and LS_ERR_NONFINITE goes to *status_dev (nullable).
 */
ls_status_t ls_lse_merge(int32_t num_parts, int64_t rows, int32_t dim_v,
                         const float* o_part, const float* lse_part,
                         void* o_bf16, float* o_f32, float* lse, int32_t* status_dev, void* stream);

/*
 * The same merge with the numerator carried the way the paper's production run exchanges it
 * (Sec. "Global Full-Attention Forward Composition", last paragraph: n_t is reduced in BF16,
 * the maximum, the denominator and the global LSE stay FP32): every shard's term
 * e^{l_r-m} o_r is rounded to bf16 and the terms are added in shard order with a bf16
 * running sum; o = n/a from that n.  Same arguments, layouts and status rules as
 * ls_lse_merge; lse is identical to ls_lse_merge's.
 */
ls_status_t ls_lse_merge_bf16_numerator(int32_t num_parts, int64_t rows, int32_t dim_v,
                         const float* o_part, const float* lse_part,
                         void* o_bf16, float* o_f32, float* lse, int32_t* status_dev, void* stream);

/*
 * Replay forward with the merge folded in: the composed output of Eq. qwen-global-attn and
 * its log-normaliser, without the per-shard partials ever reaching memory.  This is the
 * form of the score-only passes of a group member (old and reference scoring keep no
 * per-shard state, Sec. "Four-Block Response Replay") and of every block of a blockwise
 * replay.  The partials are the response block, every prefix shard (sub-range by
 * sub-range) and every appended suffix block; the CTAs that own a row tile fold them into
 * o_f32 / lse in that fixed order with the pairwise form of Eq. qwen-lse-parts
 * (m = max(l, l_r); a = e^{l-m} + e^{l_r-m}; o = (e^{l-m} o + e^{l_r-m} o_r)/a; l = m + log a),
 * so the result is bit-reproducible; the last one also writes o_bf16.
 *  Response query t sits at global position P + T + t (T = suffix tokens) and sees all P
 *  prefix positions, all T suffix positions and the response positions j <= t.
 *  q [R,Hq,dim_k], k_resp [R,Hkv,dim_k], v_resp [R,Hkv,dim_v] bf16
 *  o_bf16 [R,Hq,dim_v] bf16 (nullable); o_f32 [R,Hq,dim_v] fp32 (required: it is the running
 *  value; the backward consumes it); lse [R,Hq] fp32.
 *  workspace: ls_replay_attn_workspace_bytes(.., LS_WORKSPACE_FWD_MERGED) bytes (hand-over
 *  counters; for the 576/512 shape also a second running l of R*Hq floats).
 */
ls_status_t ls_replay_attn_fwd_merged(const ls_pages_t* pages, const ls_attn_params_t* prm,
                                      const void* q, const void* k_resp, const void* v_resp,
                                      void* o_bf16, float* o_f32, float* lse,
                                      void* workspace, size_t workspace_bytes,
                                      int32_t* status_dev, void* stream);

/*
 * Replay backward with the prefix detached (Sec. "Lazy Gradient Pages"):
 *   Delta = dO.O; p_tj = exp(s_tj - LSE); ds_tj = p_tj (dO_th.v_j - Delta)
 *   dQ_th = scale * sum_j ds_tj k_j over prefix, suffix and response keys; the per-shard
 *           contributions are summed on the device in a fixed order (Eq. qwen-dq-reduce)
 *   dK_resp_j = scale * sum_{t>=j,h in group} ds_tj q_th;  dV_resp_j = sum p_tj dO_th
 * Prefix pages get no gradient and are not written.  With suffix blocks on the handle
 * (blockwise replay) the keys of every suffix block additionally receive
 *   dk_grad[key] += scale * sum_{t,h in group} ds_t,key q_th,  dv_grad[key] += sum p_t,key dO_th
 * in the fp32 gradient pages given to ls_suffix_pages_reserve, and LS_FLAG_ADD_SUFFIX_GRAD
 * adds the gradient pages of the block popped last to dk_resp / dv_resp.
 *  o_f32 [R,Hq,dim_v], lse [R,Hq] from ls_lse_merge / ls_replay_attn_fwd_merged;
 *  d_o [R,Hq,dim_v] bf16; dq [R,Hq,dim_k], dk_resp [R,Hkv,dim_k], dv_resp [R,Hkv,dim_v] bf16
 *  workspace: ls_replay_attn_workspace_bytes(.., LS_WORKSPACE_BWD) bytes, 16-byte aligned: one
 *  fp32 running dQ of R*Hq*dim_k, Delta and the hand-over counters; a response shorter than a
 *  Q tile adds fp32 partials of the same size (one per range of keys that a CTA walks, at most
 *  one per SM and KV head), the 576/512 shape the fp32 sums of its head and part ranges.
 */
ls_status_t ls_replay_attn_bwd(const ls_pages_t* pages, const ls_attn_params_t* prm,
                               const void* q, const void* k_resp, const void* v_resp,
                               const float* o_f32, const float* lse, const void* d_o,
                               void* dq, void* dk_resp, void* dv_resp,
                               void* workspace, size_t workspace_bytes,
                               int32_t* status_dev, void* stream);

/*
 * Response suffix as temporary pages behind the resident prefix (Sec. "Four-Block Response
 * Replay": a no-grad suffix pass appends each block's KV pages, the policy pass walks the
 * blocks in reverse and pops them; Sec. "Lazy Gradient Pages": K/V gradient pages are kept
 * for the response suffix only; Sec. "LongStraw: Long-Context Execution Design": append/pop
 * transactions with a version check at every replay boundary; Sec. "State Inventory and
 * Ownership": branches may append suffix pages but cannot mutate the shared prefix).
 *
 * ls_suffix_pages_reserve: call once before the first append.  max_blocks, max_pages bound
 * the suffix; dk_grad [max_pages, page_size, Hkv, dim_k] and dv_grad [.., dim_v] are the
 * caller-owned fp32 gradient pages, indexed by suffix page SLOT (the s-th page appended and
 * not yet popped has slot s), or both NULL for forward-only use.  Allocates the handle's
 * (small) device metadata for that capacity; no later suffix call allocates.
 *
 * ls_suffix_pages_append: copies n_tokens of k_block [n,Hkv,dim_k] / v_block [n,Hkv,dim_v]
 * (bf16, device) into ceil(n/page_size) pool pages phys_pages[] (host array), which must be
 * distinct, inside the pool and mapped neither by the prefix nor by the suffix
 * (LS_ERR_BAD_PAGE_TABLE); the unused tail of the last page is zero-filled and the block's
 * gradient pages are zeroed.  With v_aliases_k, v_block is ignored.  Every block starts on a
 * fresh page.  Enqueued on `stream`; later attention calls on the same stream see the block.
 *
 * ls_suffix_pages_pop: unmaps the last block (its pool pages are the caller's again; its
 * gradient pages keep their contents for LS_FLAG_ADD_SUFFIX_GRAD).  Host-only.
 *
 * Each append / pop increments ls_pages_generation (1 after build).
 * Supported for head dims 128 and 256 (LS_ERR_UNSUPPORTED_SHAPE for 576/512).
 */
ls_status_t ls_suffix_pages_reserve(ls_pages_t* pages, int32_t max_blocks, int32_t max_pages,
                                    float* dk_grad, float* dv_grad);
ls_status_t ls_suffix_pages_append(ls_pages_t* pages, int32_t n_tokens, const int32_t* phys_pages,
                                   const void* k_block, const void* v_block, void* stream);
ls_status_t ls_suffix_pages_pop(ls_pages_t* pages);
uint64_t ls_pages_generation(const ls_pages_t* pages);
int64_t ls_suffix_pages_tokens(const ls_pages_t* pages);

/*
 * Sparse (DSA) replay over the shared latent (Sec. "GLM Attention: MLA, DSA, and IndexShare",
 * Eq. dsa-index, Eq. dsa-attention; the selection is global over the logical context as
 * Eq. glm-global-dsa requires, not per shard).  For response query t:
 *   I[t,s] = sum_j w[t,j] ReLU(<q_index[t,j], k_index[s]>)          s = 0 .. P-1
 *   S_t    = the top_k prefix positions by I[t,:]; ties go to the lower position; all P when P <= top_k
 *   u_t    = softmax attention of q[t,h] over the latent rows {c_s : s in S_t} and the causal response
 *            block (j <= t, always attended: the response is short and dense), value = first dim_v
 *            channels of the latent row
 * The backward holds S_t fixed (TopK is piecewise constant): dQ over the selected rows and the
 * response block, dK / dV of the response tokens; the prefix gets no gradient.
 * Requires the 576/512 shape with v_aliases_k, one KV head, 64-channel-aligned strides, no suffix
 * blocks; num_q_heads <= 128; num_index_heads in {8,16,32,64}; index_dim 128.
 *  ki_pool  [num_phys_pages, page_size, index_dim] bf16: indexer-key pages under the SAME page table
 *           as the latent pool (strides in elements)
 *  gathered caller-owned device buffer of ls_dsa_gathered_bytes() bytes that receives the selected
 *           latent rows of every query token ([pages of 64, 64, R, dim_k]); ls_dsa_attn_bwd reads
 *           what the last ls_dsa_attn_fwd of the plan left there
 * ls_dsa_plan_create builds two small internal page plans (allocates a few KB of device metadata).
 *  ls_dsa_index_scores: q_index [R, H_I, index_dim] bf16, w_index [R, H_I] fp32 -> scores [R, P] fp32
 *  ls_dsa_topk: scores -> sel [R, ls_dsa_selected_count()] int32, ascending positions per row
 *  ls_dsa_attn_fwd: q [R,Hq,dim_k], k_resp [R,1,dim_k], v_resp [R,1,dim_v] bf16 -> o_bf16 (nullable),
 *           o_f32 [R,Hq,dim_v], lse [R,Hq]; workspace ls_dsa_workspace_bytes(plan, LS_WORKSPACE_FWD)
 *  ls_dsa_attn_bwd: + d_o -> dq [R,Hq,dim_k], dk_resp [R,1,dim_k], dv_resp [R,1,dim_v] bf16;
 *           workspace ls_dsa_workspace_bytes(plan, LS_WORKSPACE_BWD)
 */
typedef struct ls_dsa_plan ls_dsa_plan_t;
typedef struct {
  int32_t R;                 /* response tokens */
  int32_t num_q_heads;       /* attention heads that share the latent */
  int32_t num_index_heads;   /* H_I (32 in the paper's configuration) */
  int32_t index_dim;         /* 128 */
  int32_t top_k;             /* positions kept per query (2,048 in the paper) */
  int32_t reserved;
  const void* ki_pool;
  int64_t ki_stride_page, ki_stride_tok;
  void* gathered;
} ls_dsa_desc_t;
size_t ls_dsa_gathered_bytes(const ls_pages_t* latent, const ls_dsa_desc_t* desc);
ls_status_t ls_dsa_plan_create(const ls_pages_t* latent, const ls_dsa_desc_t* desc, ls_dsa_plan_t** out);
ls_status_t ls_dsa_plan_destroy(ls_dsa_plan_t* plan);
int32_t ls_dsa_selected_count(const ls_dsa_plan_t* plan);
size_t ls_dsa_workspace_bytes(const ls_dsa_plan_t* plan, int which);
ls_status_t ls_dsa_index_scores(const ls_dsa_plan_t* plan, const void* q_index, const float* w_index,
                                float* scores, int32_t* status_dev, void* stream);
ls_status_t ls_dsa_topk(const ls_dsa_plan_t* plan, const float* scores, int32_t* sel, void* stream);
ls_status_t ls_dsa_attn_fwd(const ls_dsa_plan_t* plan, const int32_t* sel, float scale,
                            const void* q, const void* k_resp, const void* v_resp,
                            void* o_bf16, float* o_f32, float* lse,
                            void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream);
ls_status_t ls_dsa_attn_bwd(const ls_dsa_plan_t* plan, float scale,
                            const void* q, const void* k_resp, const void* v_resp,
                            const float* o_f32, const float* lse, const void* d_o,
                            void* dq, void* dk_resp, void* dv_resp,
                            void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream);

/*
 * ls_replay_attn_bwd for callers that cannot hand over scratch memory (the paper has no
 * counterpart; this is a packaging variant, the arithmetic and the outputs are those of
 * ls_replay_attn_bwd).  A replay scheduler that has sized the page pool to fill the GPU, or
 * code running under a framework whose allocator already owns all device memory, has
 * nowhere to take a workspace from at backward time: a late cudaMalloc there can fail or
 * stall the whole device.  This call therefore allocates nothing, in the library or in
 * CUDA: Delta, the hand-over counters and the fp32 running dQ go to a fixed array of
 * LS_STATIC_SCRATCH_BYTES that is part of the library's device image, so every GPU that
 * loads the library holds that much memory until the process exits.
 *  - Shapes whose backward workspace (ls_replay_attn_workspace_bytes) exceeds
 *    LS_STATIC_SCRATCH_BYTES are rejected with LS_ERR_WORKSPACE before any launch.
 *  - The first call on each device looks up the array's device address (the device must be
 *    current); make that first call before starting any stream capture.
 *  - All calls on a device share the one array, which keeps the previous call's contents.
 *    The call clears what must start at zero (the hand-over counters, by a memset on
 *    `stream`); every other word is written before it is read.  Two calls whose kernels
 *    overlap on the GPU (different streams) race on the array: serialise them.
 *  - The handle must belong to the current device (LS_ERR_STALE otherwise).
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
