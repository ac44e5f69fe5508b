// Host-side internals shared by the translation units of the library.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <vector>

#include "ls.h"

// Diagnostic builds only (-DLS_TIMING): flag bits in ls_attn_params_t::flags that skip one
// pipeline stage (operand loads, tensor-core instructions, per-row arithmetic) while keeping
// every barrier hand-off, so the cost of the remaining stages can be timed.  Outputs are
// meaningless when one is set.  A regular build ignores these bits.
#define LS_DBG_ABLATE_LOADS   (1 << 16)
#define LS_DBG_ABLATE_MMA     (1 << 17)
#define LS_DBG_ABLATE_SOFTMAX (1 << 18)
#define LS_DBG_ABLATE_MASK    (7 << 16)

namespace ls {

// One cached TMA descriptor of the page pool: K (which = 0) or V (1) viewed as
// (64 channels, token, 64-channel group, head, page) with a box of 64 x box_tok x box_groups;
// tail = token extent bounded to the valid tokens of the partially filled last logical page.
struct PoolMapEntry {
  int which, box_tok, box_groups, tail;
  CUtensorMap map;
};

// One block of response tokens appended behind the prefix (Sec. "Four-Block Response
// Replay"): its pages in the pool and its slot range in the gradient pages.
struct SuffixBlock {
  int32_t tokens;
  int32_t first_slot;     // first suffix page slot of the block
  int32_t num_pages;
};

// Control words of the ordered hand-over between CTAs of one launch (see ls_sm100.cuh):
// [0] ticket counter, [1] abort word, [2..3] unused, [4..] one completed-link counter per chain.
constexpr int kChainHeaderInts = 4;

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
  // drift apart.  The kernels walk S * fine prefix parts (then one part per appended suffix
  // block) and fold them back in a fixed order.
  int32_t fine;
  std::vector<int32_t> fine_page_offset;      // [S * fine + 1]
  std::vector<int64_t> fine_tokens;           // [S * fine]
  std::vector<int32_t> fine_tail_slot;        // [S * fine]

  // Response suffix (blocks appended behind the prefix; they live in pool pages that the
  // prefix does not map).  Device arrays are sized for the reserved capacity.
  int32_t suffix_cap_pages, suffix_cap_blocks;
  std::vector<ls::SuffixBlock> suffix_blocks;
  std::vector<int32_t> suffix_phys;           // physical page of every suffix page slot in use
  int64_t suffix_tokens;
  float* dk_grad;                              // caller-owned fp32 gradient pages (may be NULL)
  float* dv_grad;
  uint64_t generation;                         // bumped by every append / pop

  bool on_device;
  int device;
  int32_t* d_part_pages;         // [Np + suffix_cap_pages] physical ids: prefix (shard-local order), then suffix slots
  int32_t* d_part_page_offset;   // [S * fine + suffix_cap_blocks + 1]
  int32_t* d_part_tail_slot;     // [S * fine + suffix_cap_blocks]
  int64_t* d_part_tokens;        // [S * fine + suffix_cap_blocks]
  int32_t* d_page_table;         // [Np]

  mutable std::mutex map_mutex;
  mutable std::vector<ls::PoolMapEntry> map_cache;

  int prefix_parts() const { return desc.num_shards * fine; }
  int num_parts() const { return prefix_parts() + (int)suffix_blocks.size(); }   // parts the kernels walk before the response block
};

namespace ls {

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

// Diagnostic builds: device buffer of int64 words that CTA 0 of the big kernels fills with
// per-role cycle counts (NULL = off).  Set through ls_debug_timing_buffer (LS_TIMING builds only).
extern long long* g_timing_buffer;

// Rank-5 view (64 channels, token, channel group, head, page) with a box of
// 64 x box_tok x box_groups: one TMA instruction fills box_groups swizzled slabs.
ls_status_t encode_map5(CUtensorMap* out, const void* base, int64_t dim_d, int64_t dim_tok, int64_t dim_head,
                        int64_t dim_page, int64_t stride_tok, int64_t stride_head, int64_t stride_page,
                        int box_tok, int box_groups);

// Map of a dense [R, heads, dim] bf16 tensor whose box spans box_tok tokens of box_heads
// consecutive heads and one 64-channel group: fills a slab with rows (head, token).
ls_status_t encode_map_rows(CUtensorMap* out, const void* base, int64_t dim_d, int64_t R, int64_t heads,
                            int box_tok, int box_heads);

// The pool's K (which = 0) or V (which = 1) map for the given box, from the handle's cache
// (encoded on first use; the combinations the kernels of this shape use are encoded by
// ls_prefix_pages_build).
ls_status_t pool_map(CUtensorMap* out, const ls_pages* h, int which, int box_tok, int box_groups, bool tail);

// LS_OK when the handle is usable by a compute call on the current device with these
// parameters: device-resident, built on the current device, generation as the caller expects.
ls_status_t check_handle(const ls_pages* h, const ls_attn_params_t* prm);

// Sets the dynamic shared-memory limit of a kernel once per device.
template <typename K>
inline ls_status_t configure_smem(K kernel, int bytes, bool (&done)[64]) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LS_ERR_CUDA;
  if (!done[dev]) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
      return LS_ERR_CUDA;
    done[dev] = true;
  }
  return LS_OK;
}

// Backward of the shared-latent 576/512 shape (ls_bwd_mla.cu): fills dq_part (fp32, unscaled,
// [(parts+1), R, Hq, 576]; with dq_resp_only just the response block's partial, [R, Hq, 576]) and
// the bf16 dk_resp / dv_resp.
// kv_scratch: mla_kv_hsplit() * R * Hkv * 576 floats when that count exceeds 1 (NULL: no head split).
ls_status_t bwd_mla(const ls_pages* h, const ls_attn_params_t* prm, const void* q, const void* k_resp,
                    const void* v_resp, const float* lse, const float* delta, const void* d_o, float* dq_part,
                    void* dk_resp, void* dv_resp, bool dq_resp_only, float* kv_scratch, int32_t* status_dev,
                    cudaStream_t cs);
// Head ranges per key tile of the dK / dV launches of bwd_mla (a short response has too few key tiles to fill
// the GPU); 1 = no split.
int mla_kv_hsplit(const ls_pages* h, int R, int Hq);

// Prefix part of dQ for the 576/512 shape when V aliases K (ls_bwd_mla_dq.cu): CTA pairs walk the
// prefix parts, add dq_resp (fp32, unscaled, [R, Hq, 576]; NULL: none) and write the final bf16 dQ.
// How the parts are spread is mla_dq_split(): with more than one range per row block the sums meet
// either in `scratch` (count partials of R * Hq * 576 floats, then a reduce kernel) or, chained, in
// ONE running fp32 dQ -- dq_resp itself, or the first R * Hq * 576 floats of scratch when there is
// no response partial -- through the control words `ctl` (kChainHeaderInts + one per 64-row block).
// Without scratch or ctl every pair walks all parts.
ls_status_t bwd_mla_dq(const ls_pages* h, const ls_attn_params_t* prm, const void* q, const void* d_o,
                       const float* lse, const float* delta, float* dq_resp, float* scratch, int* ctl, void* dq,
                       int32_t* status_dev, cudaStream_t cs);
// count: ranges of parts per row block; chain: many row blocks -- the pairs of one range run together
// (its keys stay in L2) and the ranges fold into one running dQ in order; otherwise (few row blocks) all
// pairs run at once, each with a scratch partial.
struct MlaDqSplit {
  int count;
  bool chain;
};
MlaDqSplit mla_dq_split(const ls_pages* h, int R, int Hq);
// 64-row blocks of bwd_mla_dq for this call (one hand-over counter each).
int64_t mla_dq_blocks(const ls_pages* h, int R, int Hq);
// True when bwd_mla_dq serves this handle (576/512, V aliasing K, non-empty prefix).
bool mla_dq_fast(const ls_pages* h);

// Delta[t,h] = dO[t,h] . O[t,h] (fp32), one warp per row.
void launch_delta(const void* d_o, const float* o_f32, int64_t rows, int dv, float* delta, cudaStream_t st);

// Short-response dQ pass with one Q tile per KV group (single-CTA kernel): CTAs per KV head, each with an
// equal range of the KV head's key tiles and an fp32 partial of its own.  One CTA per SM of a B200, fewer
// when the prefix has under four key tiles per CTA.
inline int dq1_ranges(int Hkv, int64_t prefix_len) {
  const int64_t by_sms = 148 / (Hkv < 148 ? (Hkv > 0 ? Hkv : 1) : 148);
  const int64_t by_keys = prefix_len / 512 + 1;
  const int64_t r = by_sms < by_keys ? by_sms : by_keys;
  return (int)(r > 1 ? r : 1);
}

// How the (token, head) rows of one KV group (R tokens x g heads) are cut into Q tiles of at most
// tile_rows rows.  A tile covers bt consecutive tokens of bh consecutive heads; its row r is head
// r / bt, token r % bt (the order in which one TMA box of bt tokens x bh heads lands in shared
// memory).  Long responses use tiles of tile_rows tokens of one head.  A response shorter than a
// tile packs the rows of several heads into one tile whenever that needs fewer tiles, so that the
// K/V pages of the group are streamed once per tile of FULL rows instead of once per head.
struct RowTiling {
  int bt, bh, tiles_tok, tiles_head, nq_tiles;
  bool packed;
};
inline RowTiling row_tiling(int R, int g, int tile_rows) {
  RowTiling t;
  t.bt = tile_rows;
  t.bh = 1;
  t.tiles_tok = (R + tile_rows - 1) / tile_rows;
  t.tiles_head = g;
  t.packed = false;
  if (g > 1 && R < tile_rows) {
    const int bh = g < tile_rows ? g : tile_rows;
    const int bt = R < tile_rows / bh ? R : tile_rows / bh;
    const int tt = (R + bt - 1) / bt, th = (g + bh - 1) / bh;
    if (tt * th < g) {
      t.bt = bt;
      t.bh = bh;
      t.tiles_tok = tt;
      t.tiles_head = th;
      t.packed = true;
    }
  }
  t.nq_tiles = t.tiles_tok * t.tiles_head;
  return t;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int pg_shift_of(int page_size) { return page_size == 64 ? 6 : page_size == 128 ? 7 : page_size == 256 ? 8 : 9; }

}  // namespace ls
