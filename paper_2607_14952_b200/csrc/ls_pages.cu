// Host planner of the resident prefix: page table validation, shard boundaries
// (Sec. "From Logical Shards to Physical Pages"; Eq. qwen-page-owner;
// Eq. glm-tr-zigzag-pages), upload of the plan, TMA descriptors of the page pool, and
// the integrity checksum used between replays.
#include <algorithm>
#include <cstdlib>
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

ls_status_t encode_map(CUtensorMap* out, const void* base, int64_t dim_d, int64_t dim_tok,
                       int64_t dim_head, int64_t dim_page, int64_t stride_tok, int64_t stride_head,
                       int64_t stride_page, int box_tok) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return LS_ERR_CUDA;
  if (!aligned16(base)) return LS_ERR_ALIGNMENT;
  if ((stride_tok * 2) % 16 || (stride_head * 2) % 16 || (stride_page * 2) % 16) return LS_ERR_ALIGNMENT;
  cuuint64_t dims[4] = {(cuuint64_t)dim_d, (cuuint64_t)dim_tok, (cuuint64_t)dim_head, (cuuint64_t)dim_page};
  cuuint64_t strides[3] = {(cuuint64_t)stride_tok * 2, (cuuint64_t)stride_head * 2, (cuuint64_t)stride_page * 2};
  cuuint32_t box[4] = {64, (cuuint32_t)box_tok, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LS_OK : LS_ERR_CUDA;
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

ls_status_t encode_pool_map5(CUtensorMap* out, const ls_pages* h, int which, int box_tok, int box_groups,
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

static void free_device(ls_pages* h) {
  cudaFree(h->d_shard_phys_pages);
  cudaFree(h->d_shard_page_offset);
  cudaFree(h->d_shard_tail_slot);
  cudaFree(h->d_shard_tokens);
  cudaFree(h->d_page_table);
  h->d_shard_phys_pages = h->d_shard_page_offset = h->d_shard_tail_slot = h->d_page_table = nullptr;
  h->d_shard_tokens = nullptr;
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
  h->d_shard_phys_pages = h->d_shard_page_offset = h->d_shard_tail_slot = h->d_page_table = nullptr;
  h->d_shard_tokens = nullptr;

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

  // sub-shards for the kernels: aim at <= 32 MB of K+V per (KV head, sub-shard)
  {
    int64_t max_tokens = 0;
    for (int s = 0; s < S; ++s) max_tokens = std::max(max_tokens, h->shard_tokens[s]);
    const int64_t bytes_per_tok = (int64_t)(d->dim_k + (d->v_aliases_k ? 0 : d->dim_v)) * 2;
    int64_t fine = (max_tokens * bytes_per_tok + (32ll << 20) - 1) / (32ll << 20);
    if (const char* e = getenv("LS_SUBSPLIT")) fine = atoi(e);
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
  int64_t vs_page = d->v_aliases_k ? d->k_stride_page : d->v_stride_page;
  int64_t vs_tok = d->v_aliases_k ? d->k_stride_tok : d->v_stride_tok;
  int64_t vs_head = d->v_aliases_k ? d->k_stride_head : d->v_stride_head;
  if (!vbase) {
    delete h;
    return LS_ERR_INVALID_ARG;
  }
  if (!ls::aligned16(d->k_pool) || !ls::aligned16(vbase)) {
    delete h;
    return LS_ERR_ALIGNMENT;
  }
  const int64_t nphys = std::max<int64_t>(d->num_phys_pages, 1);
  for (int bi = 0; bi < ls::kNumBoxSizes; ++bi) {
    int bt = ls::kBoxTok[bi];
    if (bt > pg) bt = (int)pg;
    int64_t tail_tok = h->last_valid > 0 ? h->last_valid : pg;
    ls_status_t st = ls::encode_map(&h->k_maps.full[bi], d->k_pool, d->dim_k, pg, d->num_kv_heads, nphys,
                                    d->k_stride_tok, d->k_stride_head, d->k_stride_page, bt);
    if (st == LS_OK)
      st = ls::encode_map(&h->k_maps.tail[bi], d->k_pool, d->dim_k, tail_tok, d->num_kv_heads, nphys,
                          d->k_stride_tok, d->k_stride_head, d->k_stride_page, bt);
    if (st == LS_OK)
      st = ls::encode_map(&h->v_maps.full[bi], vbase, d->dim_v, pg, d->num_kv_heads, nphys, vs_tok, vs_head,
                          vs_page, bt);
    if (st == LS_OK)
      st = ls::encode_map(&h->v_maps.tail[bi], vbase, d->dim_v, tail_tok, d->num_kv_heads, nphys, vs_tok,
                          vs_head, vs_page, bt);
    if (st != LS_OK) {
      delete h;
      return st;
    }
  }

  cudaError_t e = cudaGetDevice(&h->device);
  if (e == cudaSuccess) e = ls::upload(&h->d_shard_phys_pages, h->shard_phys_pages);
  if (e == cudaSuccess) e = ls::upload(&h->d_shard_page_offset, h->fine_page_offset);
  if (e == cudaSuccess) e = ls::upload(&h->d_shard_tail_slot, h->fine_tail_slot);
  if (e == cudaSuccess) e = ls::upload(&h->d_shard_tokens, h->fine_tokens);
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

namespace ls {
ProfileSlot g_profile[LS_KERNEL_COUNT] = {};
}

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
