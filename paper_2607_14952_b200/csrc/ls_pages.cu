// Host planner of the resident prefix: page table validation, shard boundaries
// (Sec. "From Logical Shards to Physical Pages"; Eq. qwen-page-owner;
// Eq. glm-tr-zigzag-pages), upload of the plan, TMA descriptors of the page pool, and
// the integrity checksum used between replays.
#include <algorithm>
#include <mutex>
#include <new>

#include "ls_internal.h"
#include "ls_sm100.cuh"

namespace ls {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

ls_status_t encode_map5(CUtensorMap* out, const void* base, int64_t dim_d, int64_t dim_tok, int64_t dim_head,
                        int64_t dim_page, int64_t stride_tok, int64_t stride_head, int64_t stride_page,
                        int box_tok, int box_groups) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return LS_ERR_CUDA;
  if (!aligned16(base)) return LS_ERR_ALIGNMENT;
  if ((stride_tok * 2) % 16 || (stride_head * 2) % 16 || (stride_page * 2) % 16 || dim_d % 64) return LS_ERR_ALIGNMENT;
  cuuint64_t dims[5] = {64, (cuuint64_t)dim_tok, (cuuint64_t)(dim_d / 64), (cuuint64_t)dim_head,
                        (cuuint64_t)dim_page};
  cuuint64_t strides[4] = {(cuuint64_t)stride_tok * 2, 128, (cuuint64_t)stride_head * 2,
                           (cuuint64_t)stride_page * 2};
  cuuint32_t box[5] = {64, (cuuint32_t)box_tok, (cuuint32_t)box_groups, 1, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LS_OK : LS_ERR_CUDA;
}

ls_status_t encode_map_rows(CUtensorMap* out, const void* base, int64_t dim_d, int64_t R, int64_t heads,
                            int box_tok, int box_heads) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return LS_ERR_CUDA;
  if (!aligned16(base) || dim_d % 64) return LS_ERR_ALIGNMENT;
  cuuint64_t dims[5] = {64, (cuuint64_t)R, (cuuint64_t)(dim_d / 64), (cuuint64_t)heads, 1};
  cuuint64_t strides[4] = {(cuuint64_t)(heads * dim_d * 2), 128, (cuuint64_t)(dim_d * 2),
                           (cuuint64_t)(R * heads * dim_d * 2)};
  cuuint32_t box[5] = {64, (cuuint32_t)box_tok, 1, (cuuint32_t)box_heads, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LS_OK : LS_ERR_CUDA;
}

static ls_status_t encode_pool_map5(CUtensorMap* out, const ls_pages* h, int which, int box_tok, int box_groups,
                                    bool tail) {
  const ls_pages_desc_t& d = h->desc;
  const bool v = which == 1;
  const bool alias = v && d.v_aliases_k;
  const void* base = (v && !alias) ? d.v_pool : d.k_pool;
  const int64_t s_tok = (v && !alias) ? d.v_stride_tok : d.k_stride_tok;
  const int64_t s_head = (v && !alias) ? d.v_stride_head : d.k_stride_head;
  const int64_t s_page = (v && !alias) ? d.v_stride_page : d.k_stride_page;
  const int64_t dim = v ? d.dim_v : d.dim_k;
  const int64_t tok = tail && h->last_valid > 0 ? h->last_valid : d.page_size;
  return encode_map5(out, base, dim, tok, d.num_kv_heads, std::max<int64_t>(d.num_phys_pages, 1), s_tok, s_head,
                     s_page, std::min<int>(box_tok, d.page_size), box_groups);
}

ls_status_t pool_map(CUtensorMap* out, const ls_pages* h, int which, int box_tok, int box_groups, bool tail) {
  std::lock_guard<std::mutex> lock(h->map_mutex);
  for (const PoolMapEntry& e : h->map_cache)
    if (e.which == which && e.box_tok == box_tok && e.box_groups == box_groups && e.tail == (int)tail) {
      *out = e.map;
      return LS_OK;
    }
  PoolMapEntry e;
  e.which = which;
  e.box_tok = box_tok;
  e.box_groups = box_groups;
  e.tail = tail;
  const ls_status_t st = encode_pool_map5(&e.map, h, which, box_tok, box_groups, tail);
  if (st != LS_OK) return st;
  h->map_cache.push_back(e);
  *out = e.map;
  return LS_OK;
}

ls_status_t check_handle(const ls_pages* h, const ls_attn_params_t* prm) {
  if (!h || !prm) return LS_ERR_INVALID_ARG;
  if (!h->on_device) return LS_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return LS_ERR_CUDA;
  if (dev != h->device) return LS_ERR_STALE;
  if (prm->generation != 0 && prm->generation != h->generation) return LS_ERR_STALE;
  return LS_OK;
}

static void even_chunks(int64_t n, int64_t parts, std::vector<int64_t>& bounds) {
  bounds.assign(parts + 1, 0);
  int64_t base = n / parts, rem = n % parts;
  for (int64_t c = 0; c < parts; ++c) bounds[c + 1] = bounds[c] + base + (c < rem ? 1 : 0);
}

static bool shape_supported(int dk, int dv) {
  return (dk == 128 && dv == 128) || (dk == 256 && dv == 256) || (dk == 576 && dv == 512);
}

template <typename T>
static cudaError_t upload(T** dst, const std::vector<T>& src) {
  size_t bytes = std::max<size_t>(src.size(), 1) * sizeof(T);
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(dst), bytes);
  if (e != cudaSuccess) return e;
  if (!src.empty()) e = cudaMemcpy(*dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice);
  return e;
}

static void free_part_arrays(ls_pages* h) {
  cudaFree(h->d_part_pages);
  cudaFree(h->d_part_page_offset);
  cudaFree(h->d_part_tail_slot);
  cudaFree(h->d_part_tokens);
  h->d_part_pages = h->d_part_page_offset = h->d_part_tail_slot = nullptr;
  h->d_part_tokens = nullptr;
}

static void free_device(ls_pages* h) {
  free_part_arrays(h);
  cudaFree(h->d_page_table);
  h->d_page_table = nullptr;
}

// (Re)creates the device arrays that describe the parts the kernels walk -- prefix sub-shards,
// then one part per suffix block -- with room for the reserved suffix capacity.
static cudaError_t upload_part_arrays(ls_pages* h) {
  const int64_t Np = h->num_logical_pages;
  const int np = h->prefix_parts();
  std::vector<int32_t> pages(h->shard_phys_pages);
  pages.resize(Np + h->suffix_cap_pages, 0);
  std::vector<int32_t> off(h->fine_page_offset);
  off.resize(np + h->suffix_cap_blocks + 1, (int32_t)Np);
  std::vector<int32_t> tail(h->fine_tail_slot);
  tail.resize(np + h->suffix_cap_blocks, -1);
  std::vector<int64_t> toks(h->fine_tokens);
  toks.resize(np + h->suffix_cap_blocks, 0);
  free_part_arrays(h);
  cudaError_t e = upload(&h->d_part_pages, pages);
  if (e == cudaSuccess) e = upload(&h->d_part_page_offset, off);
  if (e == cudaSuccess) e = upload(&h->d_part_tail_slot, tail);
  if (e == cudaSuccess) e = upload(&h->d_part_tokens, toks);
  return e;
}

}  // namespace ls

extern "C" ls_status_t ls_prefix_pages_build(const ls_pages_desc_t* d, const int32_t* phys_of_logical,
                                             ls_pages_t** out) {
  if (out) *out = nullptr;
  if (!d || !out) return LS_ERR_INVALID_ARG;
  if (d->prefix_len < 0 || d->num_shards < 1 || d->num_kv_heads < 1 || d->num_phys_pages < 0)
    return LS_ERR_INVALID_ARG;
  if (d->shard_policy < LS_SHARD_CONTIGUOUS || d->shard_policy > LS_SHARD_ZIGZAG) return LS_ERR_INVALID_ARG;
  if (!(d->page_size == 64 || d->page_size == 128 || d->page_size == 256 || d->page_size == 512))
    return LS_ERR_UNSUPPORTED_SHAPE;
  if (!ls::shape_supported(d->dim_k, d->dim_v)) return LS_ERR_UNSUPPORTED_SHAPE;
  if (d->v_aliases_k && d->dim_v > d->dim_k) return LS_ERR_UNSUPPORTED_SHAPE;
  const int64_t pg = d->page_size;
  const int64_t Np = (d->prefix_len + pg - 1) / pg;
  if (Np > d->num_phys_pages || Np > INT32_MAX) return LS_ERR_INVALID_ARG;
  const int S = d->num_shards;

  ls_pages* h = new (std::nothrow) ls_pages();
  if (!h) return LS_ERR_INVALID_ARG;
  h->desc = *d;
  h->num_logical_pages = Np;
  h->last_valid = d->prefix_len == 0 ? 0 : (int32_t)(d->prefix_len - (Np - 1) * pg);
  h->on_device = false;
  h->device = -1;
  h->d_part_pages = h->d_part_page_offset = h->d_part_tail_slot = h->d_page_table = nullptr;
  h->d_part_tokens = nullptr;
  h->suffix_cap_pages = h->suffix_cap_blocks = 0;
  h->suffix_tokens = 0;
  h->dk_grad = h->dv_grad = nullptr;
  h->generation = 1;

  // page table: one-to-one into the pool
  h->page_table.resize(Np);
  {
    std::vector<uint8_t> seen(d->num_phys_pages, 0);
    for (int64_t p = 0; p < Np; ++p) {
      int64_t phys = phys_of_logical ? phys_of_logical[p] : p;
      if (phys < 0 || phys >= d->num_phys_pages || seen[phys]) {
        delete h;
        return LS_ERR_BAD_PAGE_TABLE;
      }
      seen[phys] = 1;
      h->page_table[p] = (int32_t)phys;
    }
  }

  // shard plan
  h->shard_of_page.assign(Np, 0);
  h->shard_page_offset.assign(S + 1, 0);
  h->shard_logical_pages.clear();
  h->shard_logical_pages.reserve(Np);
  std::vector<int64_t> b;
  for (int s = 0; s < S; ++s) {
    if (d->shard_policy == LS_SHARD_CONTIGUOUS) {
      if (s == 0) ls::even_chunks(Np, S, b);
      for (int64_t p = b[s]; p < b[s + 1]; ++p) h->shard_logical_pages.push_back((int32_t)p);
    } else if (d->shard_policy == LS_SHARD_CYCLIC) {
      for (int64_t p = s; p < Np; p += S) h->shard_logical_pages.push_back((int32_t)p);
    } else {
      if (s == 0) ls::even_chunks(Np, 2 * (int64_t)S, b);
      int m = 2 * S - 1 - s;
      for (int64_t p = b[s]; p < b[s + 1]; ++p) h->shard_logical_pages.push_back((int32_t)p);
      for (int64_t p = b[m]; p < b[m + 1]; ++p) h->shard_logical_pages.push_back((int32_t)p);
    }
    h->shard_page_offset[s + 1] = (int64_t)h->shard_logical_pages.size();
  }
  h->shard_phys_pages.resize(Np);
  h->shard_tokens.assign(S, 0);
  h->shard_tail_slot.assign(S, -1);
  for (int s = 0; s < S; ++s) {
    int64_t lo = h->shard_page_offset[s], hi = h->shard_page_offset[s + 1];
    int64_t tokens = (hi - lo) * pg;
    for (int64_t i = lo; i < hi; ++i) {
      int32_t p = h->shard_logical_pages[i];
      h->shard_of_page[p] = s;
      h->shard_phys_pages[i] = h->page_table[p];
      if (p == Np - 1 && h->last_valid != pg) {
        tokens -= pg - h->last_valid;
        h->shard_tail_slot[s] = (int32_t)(i - lo);
      }
    }
    h->shard_tokens[s] = tokens;
  }

  // sub-shards for the kernels: aim at <= stream_budget_kib (default 32 MB) of K+V per
  // (KV head, sub-shard), at most 16 per shard
  {
    int64_t max_tokens = 0;
    for (int s = 0; s < S; ++s) max_tokens = std::max(max_tokens, h->shard_tokens[s]);
    const int64_t bytes_per_tok = (int64_t)(d->dim_k + (d->v_aliases_k ? 0 : d->dim_v)) * 2;
    const int64_t budget = (d->stream_budget_kib > 0 ? (int64_t)d->stream_budget_kib : 32768ll) << 10;
    int64_t fine = (max_tokens * bytes_per_tok + budget - 1) / budget;
    fine = std::max<int64_t>(1, std::min<int64_t>(fine, 16));
    h->fine = (int32_t)fine;
    h->fine_page_offset.assign(S * fine + 1, 0);
    h->fine_tokens.assign(S * fine, 0);
    h->fine_tail_slot.assign(S * fine, -1);
    std::vector<int64_t> cut;
    for (int s = 0; s < S; ++s) {
      const int64_t lo = h->shard_page_offset[s], n = h->shard_page_offset[s + 1] - lo;
      ls::even_chunks(n, fine, cut);
      for (int64_t f = 0; f < fine; ++f) {
        const int64_t i = s * fine + f;
        h->fine_page_offset[i] = (int32_t)(lo + cut[f]);
        h->fine_page_offset[i + 1] = (int32_t)(lo + cut[f + 1]);
        int64_t tokens = (cut[f + 1] - cut[f]) * pg;
        const int32_t tail = h->shard_tail_slot[s];
        if (tail >= cut[f] && tail < cut[f + 1]) {
          tokens -= pg - h->last_valid;
          h->fine_tail_slot[i] = (int32_t)(tail - cut[f]);
        }
        h->fine_tokens[i] = tokens;
      }
    }
  }

  if (d->k_pool == nullptr) {   // host-only plan
    *out = h;
    return LS_OK;
  }

  const void* vbase = d->v_aliases_k ? d->k_pool : d->v_pool;
  if (!vbase) {
    delete h;
    return LS_ERR_INVALID_ARG;
  }
  if (!ls::aligned16(d->k_pool) || !ls::aligned16(vbase)) {
    delete h;
    return LS_ERR_ALIGNMENT;
  }
  // the pool's TMA descriptors for every box the kernels of this shape use
  {
    const bool mla = d->dim_k == 576;
    const bool small_pages = pg == 64;
    struct Box { int which, tok, groups; };
    std::vector<Box> boxes;
    if (mla) {
      boxes = {{0, small_pages ? 64 : 128, 1}, {1, 32, 4}, {0, 64, 1}, {0, 64, 2}, {1, 64, 1}};
    } else if (d->dim_k == 256) {
      boxes = {{0, 64, 2}, {1, 64, 2}, {0, small_pages ? 64 : 128, 1}, {1, small_pages ? 64 : 128, 1},
               {0, small_pages ? 64 : 128, small_pages ? 1 : 2}, {1, 64, 4}, {1, small_pages ? 64 : 128, small_pages ? 1 : 2}};
    } else {
      boxes = {{0, small_pages ? 64 : 128, 1}, {1, 64, 2}, {0, 64, 2}, {1, small_pages ? 64 : 128, 1},
               {0, small_pages ? 64 : 128, small_pages ? 1 : 2}, {1, small_pages ? 64 : 128, small_pages ? 1 : 2}};
    }
    CUtensorMap tmp;
    for (const Box& b : boxes)
      for (int tail = 0; tail < 2; ++tail) {
        const ls_status_t st = ls::pool_map(&tmp, h, b.which, b.tok, b.groups, tail != 0);
        if (st != LS_OK) {
          delete h;
          return st;
        }
      }
  }

  cudaError_t e = cudaGetDevice(&h->device);
  if (e == cudaSuccess) e = ls::upload_part_arrays(h);
  if (e == cudaSuccess) e = ls::upload(&h->d_page_table, h->page_table);
  if (e != cudaSuccess) {
    ls::free_device(h);
    delete h;
    return LS_ERR_CUDA;
  }
  h->on_device = true;
  *out = h;
  return LS_OK;
}

extern "C" ls_status_t ls_prefix_pages_export(const ls_pages_t* h, int32_t* page_table, int32_t* shard_of_page,
                                              int64_t* shard_page_offset, int32_t* shard_logical_pages,
                                              int64_t* shard_tokens) {
  if (!h) return LS_ERR_INVALID_ARG;
  if (page_table) std::copy(h->page_table.begin(), h->page_table.end(), page_table);
  if (shard_of_page) std::copy(h->shard_of_page.begin(), h->shard_of_page.end(), shard_of_page);
  if (shard_page_offset) std::copy(h->shard_page_offset.begin(), h->shard_page_offset.end(), shard_page_offset);
  if (shard_logical_pages)
    std::copy(h->shard_logical_pages.begin(), h->shard_logical_pages.end(), shard_logical_pages);
  if (shard_tokens) std::copy(h->shard_tokens.begin(), h->shard_tokens.end(), shard_tokens);
  return LS_OK;
}

extern "C" ls_status_t ls_prefix_pages_destroy(ls_pages_t* h) {
  if (!h) return LS_OK;
  if (h->on_device) ls::free_device(h);
  delete h;
  return LS_OK;
}

// ---------------------------------------------------------------------------------
// Checksum: sum over every element of every mapped page of (bits + 1) * odd(hash(logical
// element index)) modulo 2^64.  Integer addition commutes, so the 64-bit atomic sum is
// deterministic; the position-dependent multiplier makes swaps and moves visible.
// ---------------------------------------------------------------------------------
namespace ls {

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__global__ void checksum_kernel(const uint16_t* __restrict__ pool, const int32_t* __restrict__ page_table,
                                int64_t num_pages, int pg, int heads, int dim, int64_t s_page, int64_t s_tok,
                                int64_t s_head, uint64_t salt, unsigned long long* out) {
  const int64_t per_page = (int64_t)pg * heads * dim;
  const int64_t total = num_pages * per_page;
  uint64_t acc = 0;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int64_t p = i / per_page, r = i % per_page;
    int tok = (int)(r / ((int64_t)heads * dim));
    int rem = (int)(r % ((int64_t)heads * dim));
    int hd = rem / dim, c = rem % dim;
    uint16_t bits = pool[(int64_t)page_table[p] * s_page + (int64_t)tok * s_tok + (int64_t)hd * s_head + c];
    acc += ((uint64_t)bits + 1) * (mix64((uint64_t)i ^ salt) | 1ull);
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0 && acc) atomicAdd(out, (unsigned long long)acc);
}

}  // namespace ls

extern "C" ls_status_t ls_prefix_pages_checksum(const ls_pages_t* h, uint64_t* scratch_dev, uint64_t* out,
                                                void* stream) {
  if (!h || !scratch_dev || !out) return LS_ERR_INVALID_ARG;
  if (!h->on_device) return LS_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return LS_ERR_CUDA;
  if (dev != h->device) return LS_ERR_STALE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const ls_pages_desc_t& d = h->desc;
  if (cudaMemsetAsync(scratch_dev, 0, sizeof(uint64_t), st) != cudaSuccess) return LS_ERR_CUDA;
  if (h->num_logical_pages > 0) {
    int blocks = 148 * 8;
    ls::checksum_kernel<<<blocks, 256, 0, st>>>(static_cast<const uint16_t*>(d.k_pool), h->d_page_table,
                                               h->num_logical_pages, d.page_size, d.num_kv_heads, d.dim_k,
                                               d.k_stride_page, d.k_stride_tok, d.k_stride_head, 0x4b,
                                               reinterpret_cast<unsigned long long*>(scratch_dev));
    if (!d.v_aliases_k)
      ls::checksum_kernel<<<blocks, 256, 0, st>>>(static_cast<const uint16_t*>(d.v_pool), h->d_page_table,
                                                 h->num_logical_pages, d.page_size, d.num_kv_heads, d.dim_v,
                                                 d.v_stride_page, d.v_stride_tok, d.v_stride_head, 0x56,
                                                 reinterpret_cast<unsigned long long*>(scratch_dev));
  }
  if (cudaMemcpyAsync(out, scratch_dev, sizeof(uint64_t), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return LS_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return LS_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

// ---------------------------------------------------------------------------------
// Response suffix as temporary pages (Sec. "Four-Block Response Replay"): append copies one
// block of response K/V into pool pages the prefix does not map, pop unmaps the last block.
// ---------------------------------------------------------------------------------
namespace ls {

// Copies a dense [n, heads, dim] bf16 block into pool pages (16 bytes per thread step) and
// zero-fills the rest of the last page.  slot_pages: physical ids of the block's pages.
__global__ void suffix_copy_kernel(const uint4* __restrict__ src, uint16_t* __restrict__ pool,
                                   const int32_t* __restrict__ slot_pages, int n_tokens, int num_pages, int pg,
                                   int heads, int dim, int64_t s_page, int64_t s_tok, int64_t s_head) {
  const int vec_per_tok = heads * dim / 8;
  const int64_t total = (int64_t)num_pages * pg * vec_per_tok;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t tok = i / vec_per_tok;
    const int r = (int)(i % vec_per_tok);
    const int hd = (r * 8) / dim, c = (r * 8) % dim;
    const uint4 v = tok < n_tokens ? src[i] : make_uint4(0u, 0u, 0u, 0u);
    uint16_t* dst = pool + (int64_t)slot_pages[tok / pg] * s_page + (tok % pg) * s_tok + (int64_t)hd * s_head + c;
    *reinterpret_cast<uint4*>(dst) = v;
  }
}

}  // namespace ls

extern "C" ls_status_t ls_suffix_pages_reserve(ls_pages_t* h, int32_t max_blocks, int32_t max_pages, float* dk_grad,
                                               float* dv_grad) {
  if (!h || max_blocks < 0 || max_pages < 0 || max_blocks > 4096) return LS_ERR_INVALID_ARG;
  if (!h->on_device || !h->suffix_blocks.empty()) return LS_ERR_INVALID_ARG;
  if ((dk_grad == nullptr) != (dv_grad == nullptr)) return LS_ERR_INVALID_ARG;
  if (h->desc.dim_k == 576) return LS_ERR_UNSUPPORTED_SHAPE;
  if (!ls::aligned16(dk_grad) || !ls::aligned16(dv_grad)) return LS_ERR_ALIGNMENT;
  if (h->num_logical_pages + max_pages > h->desc.num_phys_pages) return LS_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return LS_ERR_CUDA;
  if (dev != h->device) return LS_ERR_STALE;
  h->suffix_cap_blocks = max_blocks;
  h->suffix_cap_pages = max_pages;
  h->dk_grad = dk_grad;
  h->dv_grad = dv_grad;
  if (cudaDeviceSynchronize() != cudaSuccess) return LS_ERR_CUDA;   // no kernel may still read the old arrays
  if (ls::upload_part_arrays(h) != cudaSuccess) return LS_ERR_CUDA;
  ++h->generation;
  return LS_OK;
}

extern "C" ls_status_t ls_suffix_pages_append(ls_pages_t* h, int32_t n_tokens, const int32_t* phys_pages,
                                              const void* k_block, const void* v_block, void* stream) {
  if (!h || n_tokens < 1 || !phys_pages || !k_block) return LS_ERR_INVALID_ARG;
  if (!h->on_device) return LS_ERR_INVALID_ARG;
  const ls_pages_desc_t& d = h->desc;
  if (!d.v_aliases_k && !v_block) return LS_ERR_INVALID_ARG;
  if (!ls::aligned16(k_block) || !ls::aligned16(v_block)) return LS_ERR_ALIGNMENT;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return LS_ERR_CUDA;
  if (dev != h->device) return LS_ERR_STALE;
  const int pg = d.page_size;
  const int n_pages = (n_tokens + pg - 1) / pg;
  const int first_slot = (int)h->suffix_phys.size();
  if ((int)h->suffix_blocks.size() + 1 > h->suffix_cap_blocks || first_slot + n_pages > h->suffix_cap_pages)
    return LS_ERR_INVALID_ARG;
  // the new pages must be free: in range, distinct, mapped neither by the prefix nor by the suffix
  {
    std::vector<uint8_t> used(d.num_phys_pages, 0);
    for (int32_t p : h->page_table) used[p] = 1;
    for (int32_t p : h->suffix_phys) used[p] = 1;
    for (int i = 0; i < n_pages; ++i) {
      const int64_t p = phys_pages[i];
      if (p < 0 || p >= d.num_phys_pages || used[p]) return LS_ERR_BAD_PAGE_TABLE;
      used[p] = 1;
    }
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t Np = h->num_logical_pages;
  const int part = h->prefix_parts() + (int)h->suffix_blocks.size();
  for (int i = 0; i < n_pages; ++i) h->suffix_phys.push_back(phys_pages[i]);
  ls::SuffixBlock blk;
  blk.tokens = n_tokens;
  blk.first_slot = first_slot;
  blk.num_pages = n_pages;
  h->suffix_blocks.push_back(blk);
  h->suffix_tokens += n_tokens;
  ++h->generation;
  // device plan: the block is one more part behind the prefix parts (pageable host sources: the
  // runtime stages them before returning, so the vectors may change afterwards)
  const int32_t off_end = (int32_t)(Np + first_slot + n_pages);
  const int64_t tokens64 = n_tokens;
  cudaError_t e = cudaMemcpyAsync(h->d_part_pages + Np + first_slot, h->suffix_phys.data() + first_slot,
                                  n_pages * sizeof(int32_t), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(h->d_part_page_offset + part + 1, &off_end, sizeof(int32_t), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(h->d_part_tokens + part, &tokens64, sizeof(int64_t), cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return LS_ERR_CUDA;
  const int32_t* slot_pages = h->d_part_pages + Np + first_slot;
  const int blocks = (int)std::min<int64_t>(((int64_t)n_pages * pg * d.num_kv_heads * d.dim_k / 8 + 255) / 256, 148 * 8);
  ls::suffix_copy_kernel<<<blocks, 256, 0, st>>>(static_cast<const uint4*>(k_block),
                                                const_cast<uint16_t*>(static_cast<const uint16_t*>(d.k_pool)),
                                                slot_pages, n_tokens, n_pages, pg, d.num_kv_heads, d.dim_k,
                                                d.k_stride_page, d.k_stride_tok, d.k_stride_head);
  if (!d.v_aliases_k)
    ls::suffix_copy_kernel<<<blocks, 256, 0, st>>>(static_cast<const uint4*>(v_block),
                                                  const_cast<uint16_t*>(static_cast<const uint16_t*>(d.v_pool)),
                                                  slot_pages, n_tokens, n_pages, pg, d.num_kv_heads, d.dim_v,
                                                  d.v_stride_page, d.v_stride_tok, d.v_stride_head);
  if (h->dk_grad) {
    const size_t per_page_k = (size_t)pg * d.num_kv_heads * d.dim_k * sizeof(float);
    const size_t per_page_v = (size_t)pg * d.num_kv_heads * d.dim_v * sizeof(float);
    e = cudaMemsetAsync(reinterpret_cast<char*>(h->dk_grad) + first_slot * per_page_k, 0, n_pages * per_page_k, st);
    if (e == cudaSuccess)
      e = cudaMemsetAsync(reinterpret_cast<char*>(h->dv_grad) + first_slot * per_page_v, 0, n_pages * per_page_v, st);
    if (e != cudaSuccess) return LS_ERR_CUDA;
  }
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

extern "C" ls_status_t ls_suffix_pages_pop(ls_pages_t* h) {
  if (!h || h->suffix_blocks.empty()) return LS_ERR_INVALID_ARG;
  const ls::SuffixBlock blk = h->suffix_blocks.back();
  h->suffix_blocks.pop_back();
  h->suffix_phys.resize(blk.first_slot);
  h->suffix_tokens -= blk.tokens;
  ++h->generation;
  return LS_OK;
}

extern "C" uint64_t ls_pages_generation(const ls_pages_t* h) { return h ? h->generation : 0; }

extern "C" int64_t ls_suffix_pages_tokens(const ls_pages_t* h) { return h ? h->suffix_tokens : 0; }

namespace ls {
ProfileSlot g_profile[LS_KERNEL_COUNT] = {};
long long* g_timing_buffer = nullptr;
}

#ifdef LS_TIMING
// Diagnostic builds only: device buffer (>= 64 int64 words) for the kernels' cycle counters.
extern "C" void ls_debug_timing_buffer(void* dev_buffer) { ls::g_timing_buffer = static_cast<long long*>(dev_buffer); }
#endif

extern "C" ls_status_t ls_profile_arm_events(int kernel, void* start_event, void* stop_event) {
  if (kernel < 0 || kernel >= LS_KERNEL_COUNT) return LS_ERR_INVALID_ARG;
  ls::g_profile[kernel].start = static_cast<cudaEvent_t>(start_event);
  ls::g_profile[kernel].stop = static_cast<cudaEvent_t>(stop_event);
  return LS_OK;
}

namespace ls {
// One thread waits on a barrier that nobody arrives at; the bounded wait gives up after
// budget_ns and the CTA reports LS_ERR_TIMEOUT exactly as the attention kernels would.
__global__ void selftest_wait_kernel(int32_t* status, uint64_t budget_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool done = mbar_wait_budget(&bar, 0, &abort_flag, budget_ns, 1000);
    if (!done && abort_flag && status) atomicExch(status, (int)LS_ERR_TIMEOUT);
  }
  __syncthreads();
}
}  // namespace ls

extern "C" ls_status_t ls_selftest_bounded_wait(int32_t* status_dev, uint64_t budget_ns, void* stream) {
  if (!status_dev || budget_ns == 0 || budget_ns > 1000000000ull) return LS_ERR_INVALID_ARG;
  ls::selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status_dev, budget_ns);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

extern "C" const char* ls_status_string(ls_status_t s) {
  switch (s) {
    case LS_OK: return "ok";
    case LS_ERR_INVALID_ARG: return "invalid argument";
    case LS_ERR_BAD_PAGE_TABLE: return "page table is not a one-to-one map into the pool";
    case LS_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case LS_ERR_ALIGNMENT: return "pointer or stride not 16-byte aligned";
    case LS_ERR_WORKSPACE: return "workspace too small";
    case LS_ERR_STALE: return "stale handle";
    case LS_ERR_CUDA: return "CUDA error";
    case LS_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case LS_ERR_NONFINITE: return "non-finite value";
    default: return "unknown status";
  }
}
