// Sparse (DSA) response replay over the shared latent (Sec. "GLM Attention: MLA, DSA, and
// IndexShare", Eq. dsa-index, Eq. dsa-attention; Eq. glm-global-dsa) for sm_100a.
//
//   I_{t,s} = sum_j w_{t,j} ReLU(<qI_{t,j}, kI_s>)        index score of prefix position s for query t
//   S_t     = TopK_s(I_{t,s}, k)                          over the WHOLE prefix, lower position wins ties
//   u_t     = Attn(q_t, {c_s : s in S_t} + the causal response block)
//
// Steps, each a kernel of this library:
//   1. index scores: a tcgen05 GEMM with the keys on the M side.  A CTA keeps the indexer queries
//      of 256 / H_I tokens (256 columns (t, j), 64 KB) resident and streams 128-key tiles of the
//      indexer-key pages through a ring; D = kI qI^T lands in TMEM (128 keys x 256 columns, two
//      buffers), and one thread per key folds its row: relu, weight, sum over the H_I heads of a
//      token -- a reduction along the thread's own registers, written coalesced along the keys.
//   2. top-k: one CTA per query row, radix select on order-preserving keys (digits of 11, 11 and 10
//      bits: three passes over the row, 16-byte loads), then an ordered pass that emits the selected
//      positions in ascending order and breaks ties at the threshold by position.  Integer work:
//      bit-exact against the rule, whatever the scheduling.
//   3. gather: the selected latent rows are copied into a pool whose "KV head" index is the query
//      token: [k / 64 pages, 64, R, 576].  On that pool the dense kernels of this library compute
//      exactly the sparse operator: KV head t = token t's selected keys, its H heads = the query
//      heads of one GQA group with one response row each.
//   4. attention: forward over the gathered pool without a response block, forward of the dense
//      causal response block, LSE merge of the two; backward: the response block's dQ partial, dK
//      and dV from the generic 576/512 kernel, then the transposed dQ kernel over the gathered pool,
//      which adds that partial and writes dQ.  The prefix gets no gradient; the selection is not
//      differentiated.
#include <cuda_bf16.h>

#include <algorithm>
#include <new>

#include "ls_internal.h"
#include "ls_sm100.cuh"

struct ls_dsa_plan {
  const ls_pages* latent;   // not owned
  ls_dsa_desc_t desc;
  int count;                // positions kept per query: min(top_k, P)
  ls_pages* gathered;       // plan over the caller's gathered buffer: KV head = query token
  ls_pages* response;       // empty-prefix plan for the dense causal response block
};

namespace ls {

// ------------------------------------------------------------------ 1. index scores
struct DsaIndexParams {
  CUtensorMap ki_map, ki_tail;   // indexer-key pages: box 64 ch x min(page, 128) tokens x 1 group
  CUtensorMap q_map;             // indexer queries as [R * H_I rows, 128]: box 64 ch x 128 rows
  const int32_t* page_table;
  const float* w;                // [R * H_I]
  float* scores;                 // [R, P]
  int32_t* status;
  long long P;
  int R, rows_total, pg_shift, n_key_tiles, tiles_per_chunk, n_blocks, num_logical_pages, num_phys_pages, last_valid;
};

constexpr int kIdxThreads = 320;          // producer warp, MMA warp, 8 fold warps (2 threads per key)
constexpr int kIdxStages = 4;
constexpr int kIdxTile = 32768;           // 128 keys x 128 channels
constexpr int kIdxB = 65536;              // 256 columns x 128 channels
constexpr int kIdxSmem = 1024 + kIdxB + kIdxStages * kIdxTile + 1024 + 512;

template <int HI>
__global__ void __launch_bounds__(kIdxThreads, 1) dsa_index_kernel(const __grid_constant__ DsaIndexParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* b_smem = smem;
  uint8_t* ring = smem + kIdxB;
  float* w_s = reinterpret_cast<float*>(ring + kIdxStages * kIdxTile);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(w_s) + 1024);
  uint64_t* b_full = bars;
  uint64_t* full = bars + 1;
  uint64_t* empty = full + kIdxStages;
  uint64_t* acc_full = empty + kIdxStages;    // [2]
  uint64_t* acc_empty = acc_full + 2;         // [2] all 256 fold threads have read the buffer
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // work item: token block (fastest, so CTAs in flight share the same keys) x chunk of key tiles
  const int block = blockIdx.x % p.n_blocks;
  const int chunk = blockIdx.x / p.n_blocks;
  const int tile0 = chunk * p.tiles_per_chunk;
  const int n_tiles = max(0, min(p.tiles_per_chunk, p.n_key_tiles - tile0));
  const int col0 = block * 256;               // first (t, j) row of the resident operand

  if (threadIdx.x == 0) {
    mbar_init(b_full, 1);
    for (int i = 0; i < kIdxStages; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], 256);
    }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (threadIdx.x >= 64) {
    const int c = threadIdx.x - 64;
    w_s[c] = (col0 + c < p.rows_total) ? p.w[col0 + c] : 0.f;
  }
  if (warp == 1) {
    tmem_alloc(tmem_holder, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    // =========================================================== producer (one thread)
    if (lane == 0 && n_tiles > 0) {
      mbar_arrive_expect_tx(b_full, kIdxB);
      for (int s = 0; s < 2; ++s)
        for (int r = 0; r < 2; ++r)
          tma_load_5d(b_smem + s * 32768 + r * 16384, &p.q_map, b_full, 0, col0 + r * 128, s, 0, 0);
      const int pg_mask = (1 << p.pg_shift) - 1;
      const int boxes = p.pg_shift == 6 ? 2 : 1;
      const int box_tok = 128 / boxes;
      uint32_t stage = 0, phase = 0, issued = 0;
      bool ok = true;
      for (int i = 0; i < n_tiles; ++i) {
        ok = ok && mbar_wait(&empty[stage], phase ^ 1, abort_flag);
        if (ok) {
          mbar_arrive_expect_tx(&full[stage], kIdxTile);
          uint8_t* dst = ring + stage * kIdxTile;
          const long long pos = (long long)(tile0 + i) * 128;
          for (int b = 0; b < boxes; ++b) {
            const long long pb = pos + b * box_tok;
            const int lp = (int)(pb >> p.pg_shift);
            // past the last page: a page coordinate beyond the pool, where TMA fills zeros
            const int page = lp < p.num_logical_pages ? __ldg(p.page_table + lp) : p.num_phys_pages;
            const bool tail = lp == p.num_logical_pages - 1 && p.last_valid != (1 << p.pg_shift);
            for (int s = 0; s < 2; ++s)
              tma_load_5d(dst + s * 16384 + b * 8192, tail ? &p.ki_tail : &p.ki_map, &full[stage], 0,
                          (int)(pb & pg_mask), s, 0, page);
          }
        }
        ++issued;
        if (++stage == (uint32_t)kIdxStages) { stage = 0; phase ^= 1; }
      }
      if (*abort_flag) {   // aborted: wait (bounded) for the copies already started
        for (uint32_t s = 0; s < (uint32_t)kIdxStages && s < issued; ++s) {
          const uint32_t last = ((issued - 1 - s) / kIdxStages) * kIdxStages + s;
          const uint64_t t_start = globaltimer_ns();
          while (!mbar_try_wait(&full[s], (last / kIdxStages) & 1, 1000) && globaltimer_ns() - t_start < 100000000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // =========================================================== MMA issuer (one thread)
    if (lane == 0 && n_tiles > 0) {
      constexpr uint32_t idesc = make_idesc(128, 256, 0, 0);
      constexpr uint32_t hi = sdesc_hi(1024);
      const uint32_t b_lo = sdesc_lo(smem_u32(b_smem), 16);
      const uint32_t ring_lo = sdesc_lo(smem_u32(ring), 16);
      uint32_t stage = 0, phase = 0;
      bool ok = mbar_wait(b_full, 0, abort_flag);
      for (int i = 0; i < n_tiles && ok; ++i) {
        const int buf = i & 1;
        if (i >= 2) {
          ok = mbar_wait(&acc_empty[buf], ((i >> 1) - 1) & 1, abort_flag);
          if (!ok) break;
        }
        ok = mbar_wait(&full[stage], phase, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_lo = ring_lo + stage * (kIdxTile >> 4);
#pragma unroll
        for (int s = 0; s < 2; ++s)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_ss(tmem_base + buf * 256, sdesc(a_lo + ((s * 16384 + k * 32) >> 4), hi),
                   sdesc(b_lo + ((s * 32768 + k * 32) >> 4), hi), idesc, (s | k) != 0);
        mma_commit(&empty[stage]);
        mma_commit(&acc_full[buf]);
        if (++stage == (uint32_t)kIdxStages) { stage = 0; phase ^= 1; }
      }
    }
  } else {
    // =========================================================== fold: one key per lane, two threads per key
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;             // which 128 of the 256 columns
    const int key = quad * 32 + lane;
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    constexpr int TPH = 128 / HI;                 // tokens per thread (HI <= 64: at least two)
    bool ok = true;
    for (int i = 0; i < n_tiles; ++i) {
      const int buf = i & 1;
      ok = __all_sync(0xffffffffu, ok && mbar_wait(&acc_full[buf], (i >> 1) & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      float acc[TPH];
#pragma unroll
      for (int t = 0; t < TPH; ++t) acc[t] = 0.f;
#pragma unroll
      for (int cg = 0; cg < 4; ++cg) {
        uint32_t d[32];
        tmem_ld32(tmem_base + lane_sel + buf * 256 + half * 128 + cg * 32, d);
        tc_wait_ld32(d);
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int c = cg * 32 + j;              // column inside this thread's half
          acc[c / HI] = fmaf(w_s[half * 128 + c], fmaxf(__uint_as_float(d[j]), 0.f), acc[c / HI]);
        }
      }
      tc_fence_before();
      mbar_arrive(&acc_empty[buf]);
      const long long pos = (long long)(tile0 + i) * 128 + key;
      if (pos < p.P) {
#pragma unroll
        for (int t = 0; t < TPH; ++t) {
          const int tok = block * (256 / HI) + half * TPH + t;
          if (tok < p.R) p.scores[(long long)tok * p.P + pos] = acc[t];
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
  if (threadIdx.x == 0 && *abort_flag && p.status) atomicExch(p.status, (int)LS_ERR_TIMEOUT);
}

template <int HI>
static ls_status_t launch_index(const DsaIndexParams& P, int grid, cudaStream_t st) {
  static bool configured[64] = {};
  const ls_status_t cs = configure_smem(dsa_index_kernel<HI>, kIdxSmem, configured);
  if (cs != LS_OK) return cs;
  dsa_index_kernel<HI><<<grid, kIdxThreads, kIdxSmem, st>>>(P);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

// ------------------------------------------------------------------ 2. top-k
// Larger float <=> larger key.
__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kTopkThreads = 1024;
constexpr int kTopkBins = 2048;            // radix digits of 11, 11 and 10 bits

// Warp 0: the digit d with  #(digit > d) < need <= #(digit >= d)  in the histogram, and #(digit > d).
// Each lane sums 64 bins, the lanes scan from the top; the lane that holds d writes the results.
__device__ __forceinline__ void topk_find_digit(const uint32_t* hist, uint32_t need, int lane, uint32_t* d_out,
                                                uint32_t* above_out) {
  constexpr int kPer = kTopkBins / 32;
  uint32_t mine = 0;
  for (int b = 0; b < kPer; ++b) mine += hist[lane * kPer + b];
  uint32_t above = 0;                                     // bins of higher lanes
  for (int l = 31; l > 0; --l) {
    const uint32_t v = __shfl_sync(0xffffffffu, mine, l);
    if (lane < l) above += v;
  }
  if (above < need && above + mine >= need) {             // exactly one lane
    uint32_t cum = above;
    int d = lane * kPer + kPer - 1;
    for (; d > lane * kPer; --d) {
      if (cum + hist[d] >= need) break;
      cum += hist[d];
    }
    *d_out = (uint32_t)d;
    *above_out = cum;
  }
}

// One histogram sweep over positions [begin, end) of a row: scores whose key, shifted down to the
// current digit, lies in [lo_full, lo_full + span] are counted under their digit.  The body runs on
// 16-byte loads (the row's first `peel` positions bring it to a 16-byte boundary), four in flight per thread.
__device__ __forceinline__ void topk_count(const float* __restrict__ s, int begin, int end, int peel, bool vec,
                                           int shift, uint32_t dmask, uint32_t lo_full, uint32_t span,
                                           uint32_t* hist, int tid) {
  auto count = [&](float f) {
    const uint32_t kh = order_key(f) >> shift;
    if (kh - lo_full <= span) atomicAdd(&hist[kh & dmask], 1u);
  };
  int body0 = begin, body1 = begin;                       // [body0, body1): whole aligned float4 groups
  if (vec) {
    body0 = begin <= peel ? peel : peel + ((begin - peel + 3) & ~3);
    body1 = body0 + (end > body0 ? ((end - body0) & ~3) : 0);
    if (body0 > end) body0 = body1 = end;
  }
  for (int i = begin + tid; i < body0; i += kTopkThreads) count(__ldg(s + i));
  const float4* s4 = reinterpret_cast<const float4*>(s + body0);
  const int n4 = (body1 - body0) >> 2;
  int i = tid;
  for (; i + 3 * kTopkThreads < n4; i += 4 * kTopkThreads) {
    const float4 a = __ldg(s4 + i), b = __ldg(s4 + i + kTopkThreads), c = __ldg(s4 + i + 2 * kTopkThreads),
                 d = __ldg(s4 + i + 3 * kTopkThreads);
    count(a.x); count(a.y); count(a.z); count(a.w);
    count(b.x); count(b.y); count(b.z); count(b.w);
    count(c.x); count(c.y); count(c.z); count(c.w);
    count(d.x); count(d.y); count(d.z); count(d.w);
  }
  for (; i < n4; i += kTopkThreads) {
    const float4 a = __ldg(s4 + i);
    count(a.x); count(a.y); count(a.z); count(a.w);
  }
  for (int j = body1 + tid; j < end; j += kTopkThreads) count(__ldg(s + j));
}

__global__ void __launch_bounds__(kTopkThreads, 2) dsa_topk_kernel(const float* __restrict__ scores, long long P64, int k,
                                                                   int32_t* __restrict__ sel) {
  const float* s = scores + (long long)blockIdx.x * P64;
  const int P = (int)P64;                                   // positions are int32
  const int count_sel = min(k, P);
  int32_t* out = sel + (long long)blockIdx.x * count_sel;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  if (P <= k) {
    for (int i = tid; i < P; i += kTopkThreads) out[i] = i;
    return;
  }
  __shared__ uint32_t hist[kTopkBins];
  __shared__ uint32_t sh_digit, sh_above;
  __shared__ uint32_t warp_gt[32], warp_eq[32];
  __shared__ uint32_t base_gt, base_eq;
  // 16-byte loads need the scores buffer on a 16-byte boundary; a row then starts 0..3 floats past one
  const bool vec = (reinterpret_cast<uintptr_t>(scores) & 15) == 0;
  const int peel = vec ? (int)((4 - (((long long)blockIdx.x * P64) & 3)) & 3) : 0;
  // ---- radix select: the key of the k-th largest score, and how many scores equal to it to take
  uint32_t prefix = 0, need = (uint32_t)k;
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 21 : pass == 1 ? 10 : 0;
    const uint32_t dmask = pass == 2 ? 1023u : 2047u;
    for (int b = tid; b < kTopkBins; b += kTopkThreads) hist[b] = 0;
    __syncthreads();
    // Pass 0 would send every score of the row through a shared-memory atomic.  Its first 64K positions
    // alone already hold `need` scores whose digit is at least some d0, so no score with a smaller digit
    // can be selected: once d0 is known the rest of the row only counts digits >= d0 (a few per cent).
    uint32_t lo = 0;
    const int head = (pass == 0 && P > 8 * 65536 && need <= 16384) ? 65536 : 0;
    if (head) {
      topk_count(s, 0, head, peel, vec, shift, dmask, 0u, dmask, hist, tid);
      __syncthreads();
      if (wid == 0) topk_find_digit(hist, need, lane, &sh_digit, &sh_above);
      __syncthreads();
      lo = sh_digit;
      __syncthreads();
    }
    topk_count(s, head, P, peel, vec, shift, dmask, (prefix >> shift) + lo, dmask - lo, hist, tid);
    __syncthreads();
    if (wid == 0) topk_find_digit(hist, need, lane, &sh_digit, &sh_above);
    __syncthreads();
    prefix |= sh_digit << shift;
    need -= sh_above;
    __syncthreads();
  }
  // ---- ordered pass: positions in ascending order; among scores equal to the threshold the lower
  // positions are taken.  A thread owns 16 consecutive positions of a 16384-position tile; it first
  // counts (greater, equal), and only a thread that owns a selected position reads its scores again.
  const uint32_t thr = prefix;
  if (tid == 0) { base_gt = 0; base_eq = 0; }
  __syncthreads();
  for (int start = 0; start < P; start += 16 * kTopkThreads) {
    const int i0 = start + 16 * tid;
    uint32_t n_gt = 0, n_eq = 0;
    if (i0 < P) {
      if (vec && i0 >= peel && ((i0 - peel) & 3) == 0 && i0 + 16 <= P) {
        const float4* s4 = reinterpret_cast<const float4*>(s + i0);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float4 v = __ldg(s4 + j);
          const uint32_t k0 = order_key(v.x), k1 = order_key(v.y), k2 = order_key(v.z), k3 = order_key(v.w);
          n_gt += (k0 > thr) + (k1 > thr) + (k2 > thr) + (k3 > thr);
          n_eq += (k0 == thr) + (k1 == thr) + (k2 == thr) + (k3 == thr);
        }
      } else {
        for (int e = 0; e < 16 && i0 + e < P; ++e) {
          const uint32_t key = order_key(__ldg(s + i0 + e));
          n_gt += key > thr;
          n_eq += key == thr;
        }
      }
    }
    uint32_t ex_gt = n_gt, ex_eq = n_eq;                     // inclusive prefix over the lanes
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t a = __shfl_up_sync(0xffffffffu, ex_gt, o), b = __shfl_up_sync(0xffffffffu, ex_eq, o);
      if (lane >= o) { ex_gt += a; ex_eq += b; }
    }
    if (lane == 31) { warp_gt[wid] = ex_gt; warp_eq[wid] = ex_eq; }
    ex_gt -= n_gt;
    ex_eq -= n_eq;
    __syncthreads();
    const uint32_t bg = base_gt, be = base_eq;
    if (n_gt | n_eq) {
      for (int w = 0; w < wid; ++w) { ex_gt += warp_gt[w]; ex_eq += warp_eq[w]; }
      uint32_t g_before = bg + ex_gt, e_before = be + ex_eq;
      for (int e = 0; e < 16 && i0 + e < P; ++e) {
        const uint32_t key = order_key(__ldg(s + i0 + e));
        const bool gt = key > thr, eq = key == thr;
        if (gt || (eq && e_before < need)) out[g_before + min(e_before, need)] = i0 + e;
        g_before += gt;
        e_before += eq;
      }
    }
    __syncthreads();
    if (tid == 0) {
      uint32_t tg = 0, te = 0;
      for (int w = 0; w < 32; ++w) { tg += warp_gt[w]; te += warp_eq[w]; }
      base_gt = bg + tg;
      base_eq = be + te;
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------ 3. gather
// gathered[(i * R + t) * dk ..] = latent row at prefix position sel[t, i] (KV head 0), 16 bytes per step
__global__ void dsa_gather_kernel(const uint16_t* __restrict__ pool, const int32_t* __restrict__ page_table,
                                  const int32_t* __restrict__ sel, int R, int count, int dk, int pg_shift,
                                  long long s_page, long long s_tok, uint16_t* __restrict__ out) {
  const int vec = dk / 8;
  const long long total = (long long)R * count * vec;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
    const int v = (int)(idx % vec);
    const long long ti = idx / vec;
    const int i = (int)(ti % count), t = (int)(ti / count);
    const int pos = sel[(long long)t * count + i];
    const uint16_t* src = pool + (long long)page_table[pos >> pg_shift] * s_page + (long long)(pos & ((1 << pg_shift) - 1)) * s_tok + v * 8;
    *reinterpret_cast<uint4*>(out + ((long long)i * R + t) * dk + v * 8) = *reinterpret_cast<const uint4*>(src);
  }
}

static size_t align16(size_t x) { return (x + 15) & ~(size_t)15; }

}  // namespace ls

// ------------------------------------------------------------------ plan
static int dsa_count(const ls_pages_t* latent, const ls_dsa_desc_t* d) {
  return (int)std::min<int64_t>(d->top_k, latent->desc.prefix_len);
}

extern "C" size_t ls_dsa_gathered_bytes(const ls_pages_t* latent, const ls_dsa_desc_t* d) {
  if (!latent || !d || d->R < 1 || d->top_k < 1) return 0;
  const int64_t pages = (dsa_count(latent, d) + 63) / 64;
  return (size_t)std::max<int64_t>(pages, 1) * 64 * d->R * latent->desc.dim_k * 2;
}

extern "C" ls_status_t ls_dsa_plan_create(const ls_pages_t* latent, const ls_dsa_desc_t* d, ls_dsa_plan_t** out) {
  if (out) *out = nullptr;
  if (!latent || !d || !out) return LS_ERR_INVALID_ARG;
  if (!latent->on_device) return LS_ERR_INVALID_ARG;
  const ls_pages_desc_t& ld = latent->desc;
  if (!(ld.dim_k == 576 && ld.dim_v == 512 && ld.v_aliases_k && ld.num_kv_heads == 1)) return LS_ERR_UNSUPPORTED_SHAPE;
  if (d->R < 1 || d->num_q_heads < 1 || d->num_q_heads > 128 || d->top_k < 1) return LS_ERR_INVALID_ARG;
  if (!(d->num_index_heads == 8 || d->num_index_heads == 16 || d->num_index_heads == 32 || d->num_index_heads == 64) ||
      d->index_dim != 128)
    return LS_ERR_UNSUPPORTED_SHAPE;
  if (ld.prefix_len < 1 || !latent->suffix_blocks.empty()) return LS_ERR_INVALID_ARG;
  if (!d->ki_pool || !d->gathered) return LS_ERR_INVALID_ARG;
  if (!ls::aligned16(d->ki_pool) || !ls::aligned16(d->gathered) || (d->ki_stride_page * 2) % 16 || (d->ki_stride_tok * 2) % 16)
    return LS_ERR_ALIGNMENT;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return LS_ERR_CUDA;
  if (dev != latent->device) return LS_ERR_STALE;
  ls_dsa_plan* p = new (std::nothrow) ls_dsa_plan();
  if (!p) return LS_ERR_INVALID_ARG;
  p->latent = latent;
  p->desc = *d;
  p->count = dsa_count(latent, d);
  p->gathered = p->response = nullptr;
  // the gathered pool: [pages of 64, 64, R "KV heads", dim_k]; KV head t holds token t's selected rows
  ls_pages_desc_t g = {};
  g.prefix_len = p->count;
  g.page_size = 64;
  g.num_shards = 1;
  g.shard_policy = LS_SHARD_CONTIGUOUS;
  g.num_kv_heads = d->R;
  g.dim_k = ld.dim_k;
  g.dim_v = ld.dim_v;
  g.v_aliases_k = 1;
  g.num_phys_pages = (p->count + 63) / 64;
  g.k_pool = d->gathered;
  g.k_stride_head = ld.dim_k;
  g.k_stride_tok = (int64_t)d->R * ld.dim_k;
  g.k_stride_page = 64 * g.k_stride_tok;
  ls_status_t st = ls_prefix_pages_build(&g, nullptr, &p->gathered);
  if (st == LS_OK) {
    // the causal response block alone: the latent's pool with an empty prefix
    ls_pages_desc_t r = ld;
    r.prefix_len = 0;
    r.num_shards = 1;
    r.shard_policy = LS_SHARD_CONTIGUOUS;
    st = ls_prefix_pages_build(&r, nullptr, &p->response);
  }
  if (st != LS_OK) {
    ls_prefix_pages_destroy(p->gathered);
    delete p;
    return st;
  }
  *out = p;
  return LS_OK;
}

extern "C" ls_status_t ls_dsa_plan_destroy(ls_dsa_plan_t* p) {
  if (!p) return LS_OK;
  ls_prefix_pages_destroy(p->gathered);
  ls_prefix_pages_destroy(p->response);
  delete p;
  return LS_OK;
}

extern "C" int32_t ls_dsa_selected_count(const ls_dsa_plan_t* p) { return p ? p->count : 0; }

extern "C" size_t ls_dsa_workspace_bytes(const ls_dsa_plan_t* p, int which) {
  if (!p) return 0;
  const size_t rows = (size_t)p->desc.R * p->desc.num_q_heads;
  const ls_pages_desc_t& ld = p->latent->desc;
  if (which == LS_WORKSPACE_FWD)      // three partials (selected prefix rows, an empty one, the response block) with their l
    return ls::align16(3 * rows * ld.dim_v * sizeof(float)) + ls::align16(3 * rows * sizeof(float));
  if (which == LS_WORKSPACE_BWD) {    // Delta, the response block's fp32 dQ partial, head-range sums of its dK / dV
    const int hsplit = ls::mla_kv_hsplit(p->response, p->desc.R, p->desc.num_q_heads);
    return ls::align16(rows * sizeof(float)) + rows * ld.dim_k * sizeof(float) +
           (hsplit > 1 ? (size_t)hsplit * p->desc.R * ld.dim_k * sizeof(float) : 0);
  }
  return 0;
}

// ------------------------------------------------------------------ entry points
extern "C" ls_status_t ls_dsa_index_scores(const ls_dsa_plan_t* p, const void* q_index, const float* w_index,
                                           float* scores, int32_t* status_dev, void* stream) {
  if (!p || !q_index || !w_index || !scores) return LS_ERR_INVALID_ARG;
  if (!ls::aligned16(q_index)) return LS_ERR_ALIGNMENT;
  const ls_pages* h = p->latent;
  const ls_pages_desc_t& ld = h->desc;
  const ls_dsa_desc_t& d = p->desc;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return LS_ERR_CUDA;
  if (dev != h->device) return LS_ERR_STALE;
  ls::DsaIndexParams P;
  const int box_tok = std::min(ld.page_size, 128);
  const int64_t tail_tok = h->last_valid > 0 ? h->last_valid : ld.page_size;
  ls_status_t st = ls::encode_map5(&P.ki_map, d.ki_pool, 128, ld.page_size, 1, std::max<int64_t>(ld.num_phys_pages, 1),
                                   d.ki_stride_tok, 128, d.ki_stride_page, box_tok, 1);
  if (st == LS_OK)
    st = ls::encode_map5(&P.ki_tail, d.ki_pool, 128, tail_tok, 1, std::max<int64_t>(ld.num_phys_pages, 1), d.ki_stride_tok,
                         128, d.ki_stride_page, box_tok, 1);
  const int64_t rows_total = (int64_t)d.R * d.num_index_heads;
  if (st == LS_OK) st = ls::encode_map5(&P.q_map, q_index, 128, rows_total, 1, 1, 128, 128, rows_total * 128, 128, 1);
  if (st != LS_OK) return st;
  P.page_table = h->d_page_table;
  P.w = w_index;
  P.scores = scores;
  P.status = status_dev;
  P.P = ld.prefix_len;
  P.R = d.R;
  P.rows_total = (int)rows_total;
  P.pg_shift = ls::pg_shift_of(ld.page_size);
  P.n_key_tiles = (int)((ld.prefix_len + 127) / 128);
  P.n_blocks = (int)((rows_total + 255) / 256);
  // enough chunks of key tiles to fill the GPU a few times over, each long enough to amortise the resident operand
  const int want_chunks = std::max(1, (148 * 4 + P.n_blocks - 1) / P.n_blocks);
  P.tiles_per_chunk = std::max(8, (P.n_key_tiles + want_chunks - 1) / want_chunks);
  const int n_chunks = (P.n_key_tiles + P.tiles_per_chunk - 1) / P.tiles_per_chunk;
  P.num_logical_pages = (int)h->num_logical_pages;
  P.num_phys_pages = (int)std::min<int64_t>(ld.num_phys_pages, INT32_MAX);
  P.last_valid = h->last_valid;
  const int64_t grid = (int64_t)n_chunks * P.n_blocks;
  if (grid > INT32_MAX) return LS_ERR_UNSUPPORTED_SHAPE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  switch (d.num_index_heads) {
    case 8: return ls::launch_index<8>(P, (int)grid, cs);
    case 16: return ls::launch_index<16>(P, (int)grid, cs);
    case 32: return ls::launch_index<32>(P, (int)grid, cs);
    default: return ls::launch_index<64>(P, (int)grid, cs);
  }
}

extern "C" ls_status_t ls_dsa_topk(const ls_dsa_plan_t* p, const float* scores, int32_t* sel, void* stream) {
  if (!p || !scores || !sel) return LS_ERR_INVALID_ARG;
  ls::dsa_topk_kernel<<<p->desc.R, ls::kTopkThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      scores, p->latent->desc.prefix_len, p->desc.top_k, sel);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

extern "C" ls_status_t ls_dsa_attn_fwd(const ls_dsa_plan_t* p, const int32_t* sel, float scale, const void* q,
                                       const void* k_resp, const void* v_resp, void* o_bf16, float* o_f32, float* lse,
                                       void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream) {
  if (!p || !sel || !q || !k_resp || !v_resp || !o_f32 || !lse) return LS_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < ls_dsa_workspace_bytes(p, LS_WORKSPACE_FWD) || !ls::aligned16(workspace))
    return LS_ERR_WORKSPACE;
  const ls_pages* h = p->latent;
  const ls_pages_desc_t& ld = h->desc;
  const ls_dsa_desc_t& d = p->desc;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const int64_t rows = (int64_t)d.R * d.num_q_heads;
  float* x_o = static_cast<float*>(workspace);
  float* x_l = reinterpret_cast<float*>(static_cast<char*>(workspace) + ls::align16(3 * rows * ld.dim_v * sizeof(float)));
  // 3. selected latent rows -> the gathered pool
  const int64_t total = (int64_t)d.R * p->count * (ld.dim_k / 8);
  ls::dsa_gather_kernel<<<(int)std::min<int64_t>((total + 255) / 256, 148 * 16), 256, 0, cs>>>(
      static_cast<const uint16_t*>(ld.k_pool), h->d_page_table, sel, d.R, p->count, ld.dim_k, ls::pg_shift_of(ld.page_size),
      ld.k_stride_page, ld.k_stride_tok, static_cast<uint16_t*>(d.gathered));
  if (cudaGetLastError() != cudaSuccess) return LS_ERR_CUDA;
  // 4a. every query token against its own selected rows: token = KV head, its heads = one GQA group, one row each
  ls_attn_params_t pg = {};
  pg.R = 1;
  pg.num_q_heads = (int32_t)rows;
  pg.scale = scale;
  pg.flags = LS_FLAG_NO_RESPONSE_BLOCK;
  ls_status_t st = ls_replay_attn_fwd(p->gathered, &pg, q, nullptr, nullptr, x_o, x_l, nullptr, 0, status_dev, stream);
  if (st != LS_OK) return st;
  // 4b. the dense causal response block (partials 1 and 2: an empty prefix partial, then the block)
  ls_attn_params_t pr = {};
  pr.R = d.R;
  pr.num_q_heads = d.num_q_heads;
  pr.scale = scale;
  st = ls_replay_attn_fwd(p->response, &pr, q, k_resp, v_resp, x_o + rows * ld.dim_v, x_l + rows, nullptr, 0, status_dev,
                          stream);
  if (st != LS_OK) return st;
  // 4c. Eq. qwen-lse-parts / qwen-global-attn over the three partials
  return ls_lse_merge(3, rows, ld.dim_v, x_o, x_l, o_bf16, o_f32, lse, status_dev, stream);
}

extern "C" ls_status_t ls_dsa_attn_bwd(const ls_dsa_plan_t* p, float scale, const void* q, const void* k_resp,
                                       const void* v_resp, const float* o_f32, const float* lse, const void* d_o, void* dq,
                                       void* dk_resp, void* dv_resp, void* workspace, size_t workspace_bytes,
                                       int32_t* status_dev, void* stream) {
  if (!p || !q || !k_resp || !v_resp || !o_f32 || !lse || !d_o || !dq || !dk_resp || !dv_resp) return LS_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < ls_dsa_workspace_bytes(p, LS_WORKSPACE_BWD) || !ls::aligned16(workspace))
    return LS_ERR_WORKSPACE;
  const void* ptrs[] = {q, k_resp, v_resp, o_f32, d_o, dq, dk_resp, dv_resp};
  for (const void* ptr : ptrs)
    if (!ls::aligned16(ptr)) return LS_ERR_ALIGNMENT;
  const ls_pages_desc_t& ld = p->latent->desc;
  const ls_dsa_desc_t& d = p->desc;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const int64_t rows = (int64_t)d.R * d.num_q_heads;
  float* delta = static_cast<float*>(workspace);
  float* dq_resp = reinterpret_cast<float*>(static_cast<char*>(workspace) + ls::align16(rows * sizeof(float)));
  ls::launch_delta(d_o, o_f32, rows, ld.dim_v, delta, cs);
  // the response block: its fp32 dQ partial, dK and dV (the only keys that receive a gradient)
  ls_attn_params_t pr = {};
  pr.R = d.R;
  pr.num_q_heads = d.num_q_heads;
  pr.scale = scale;
  float* kv_scratch = ls::mla_kv_hsplit(p->response, d.R, d.num_q_heads) > 1 ? dq_resp + rows * ld.dim_k : nullptr;
  ls_status_t st = ls::bwd_mla(p->response, &pr, q, k_resp, v_resp, lse, delta, d_o, dq_resp, dk_resp, dv_resp, true,
                               kv_scratch, status_dev, cs);
  if (st != LS_OK) return st;
  // the selected prefix rows: every (token, head) row walks its token's gathered keys, adds the response
  // block's partial and writes dQ
  ls_attn_params_t pg = {};
  pg.R = 1;
  pg.num_q_heads = (int32_t)rows;
  pg.scale = scale;
  return ls::bwd_mla_dq(p->gathered, &pg, q, d_o, lse, delta, dq_resp, nullptr, nullptr, dq, status_dev, cs);
}
