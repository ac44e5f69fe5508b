// Host-side internals shared by the translation units of the library.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <vector>

#include "ls.h"

namespace ls {

constexpr int kNumBoxSizes = 4;               // token extents of the TMA boxes we encode
constexpr int kBoxTok[kNumBoxSizes] = {16, 32, 64, 128};

inline int box_index(int tok) { return tok == 16 ? 0 : tok == 32 ? 1 : tok == 64 ? 2 : 3; }

// TMA descriptors of one bf16 pool viewed as (d, token, head, page); [box][0] covers a
// full page, [box][1] the partially filled last logical page (tokens past the valid
// count read as zero).
struct PoolMaps {
  CUtensorMap full[kNumBoxSizes];
  CUtensorMap tail[kNumBoxSizes];
};

}  // namespace ls

struct ls_pages {
  ls_pages_desc_t desc;
  int64_t num_logical_pages;   // Np
  int32_t last_valid;          // valid tokens of the last logical page (0 when P = 0)
  std::vector<int32_t> page_table;            // [Np] logical -> physical
  std::vector<int32_t> shard_of_page;         // [Np]
  std::vector<int64_t> shard_page_offset;     // [S+1]
  std::vector<int32_t> shard_logical_pages;   // [Np] shard-local order
  std::vector<int32_t> shard_phys_pages;      // [Np] physical ids in shard-local order
  std::vector<int64_t> shard_tokens;          // [S]
  // per shard: position (in its page list) of the global last logical page, or -1
  std::vector<int32_t> shard_tail_slot;       // [S]

  // Kernel-side plan: every shard is cut into `fine` contiguous sub-shards so that one
  // (KV head, sub-shard) stream of K and V fits comfortably in L2 while the CTAs that share it
  // drift apart.  The device arrays below describe the S * fine sub-shards; the kernels treat
  // them as S * fine partials and the host folds them back into the S the caller asked for.
  int32_t fine;
  std::vector<int32_t> fine_page_offset;      // [S * fine + 1]
  std::vector<int64_t> fine_tokens;           // [S * fine]
  std::vector<int32_t> fine_tail_slot;        // [S * fine]

  bool on_device;
  int device;
  int32_t* d_shard_phys_pages;   // [Np]
  int32_t* d_shard_page_offset;  // [S * fine + 1]  (sub-shards)
  int32_t* d_shard_tail_slot;    // [S * fine]
  int64_t* d_shard_tokens;       // [S * fine]
  int32_t* d_page_table;         // [Np]
  ls::PoolMaps k_maps, v_maps;
};

namespace ls {

// Encodes a rank-4 bf16 tensor map (d, token, head, page) with a 128-byte swizzle and a
// box of 64 channels x box_tok tokens.  Strides in elements.  Returns LS_OK or an error.
ls_status_t encode_map(CUtensorMap* out, const void* base, int64_t dim_d, int64_t dim_tok,
                       int64_t dim_head, int64_t dim_page, int64_t stride_tok, int64_t stride_head,
                       int64_t stride_page, int box_tok);

// One-shot event pairs armed by ls_profile_arm_events.
struct ProfileSlot {
  cudaEvent_t start, stop;
};
extern ProfileSlot g_profile[LS_KERNEL_COUNT];
inline void profile_begin(int k, cudaStream_t st) {
  if (g_profile[k].start) cudaEventRecord(g_profile[k].start, st);
}
inline void profile_end(int k, cudaStream_t st) {
  if (g_profile[k].stop) cudaEventRecord(g_profile[k].stop, st);
  g_profile[k].start = g_profile[k].stop = nullptr;
}

// Rank-5 view (64 channels, token, channel group, head, page) with a box of
// 64 x box_tok x box_groups: one TMA instruction fills box_groups swizzled slabs.
ls_status_t encode_map5(CUtensorMap* out, const void* base, int64_t dim_d, int64_t dim_tok, int64_t dim_head,
                        int64_t dim_page, int64_t stride_tok, int64_t stride_head, int64_t stride_page,
                        int box_tok, int box_groups);

// Map of a dense [R, heads, dim] bf16 tensor whose box spans box_tok tokens of box_heads
// consecutive heads and one 64-channel group: fills a slab with rows (head, token).
ls_status_t encode_map_rows(CUtensorMap* out, const void* base, int64_t dim_d, int64_t R, int64_t heads,
                            int box_tok, int box_heads);

// The pool's K (which = 0) or V (which = 1) map for the given box; tail = bounded to the valid
// tokens of the partially filled last logical page.
ls_status_t encode_pool_map5(CUtensorMap* out, const ls_pages* h, int which, int box_tok, int box_groups,
                             bool tail);

// Backward of the shared-latent 576/512 shape (ls_bwd_mla.cu): fills dq_part (fp32, unscaled,
// [(S+1), R, Hq, 576]; with dq_resp_only just the response block's partial, [R, Hq, 576]) and
// the bf16 dk_resp / dv_resp.
ls_status_t bwd_mla(const ls_pages* h, const ls_attn_params_t* prm, const void* q, const void* k_resp,
                    const void* v_resp, const float* lse, const float* delta, const void* d_o, float* dq_part,
                    void* dk_resp, void* dv_resp, bool dq_resp_only, int32_t* status_dev, cudaStream_t cs);

// Prefix part of dQ for the 576/512 shape when V aliases K (ls_bwd_mla_dq.cu): every CTA walks
// all partials, adds dq_resp (fp32, unscaled, [R, Hq, 576]) and writes the final bf16 dQ.
ls_status_t bwd_mla_dq(const ls_pages* h, const ls_attn_params_t* prm, const void* q, const void* d_o,
                       const float* lse, const float* delta, const float* dq_resp, void* dq, int32_t* status_dev,
                       cudaStream_t cs);
// True when bwd_mla_dq serves this handle (576/512, V aliasing K, non-empty prefix, LS_MLA_DQ != 0).
bool mla_dq_fast(const ls_pages* h);

// Folds `fine` consecutive sub-shard partials into each of `groups` shard partials.
ls_status_t group_merge(int groups, int fine, int64_t rows, int dv, const float* in_o, const float* in_lse,
                        float* out_o, float* out_lse, cudaStream_t st);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace ls
