// Replay backward with a detached prefix (Sec. "Lazy Gradient Pages", Eq. qwen-dq-reduce)
// for sm_100a.
//
//   Delta_th = dO_th . O_th;  p_tj = exp(s_tj - LSE_th);  ds_tj = p_tj (dO_th . v_j - Delta_th)
//   dQ_th = scale * sum_j ds_tj k_j      (prefix and response keys; per-partial sums reduced here)
//   dK_j  = scale * sum_{t>=j,h} ds_tj q_th,   dV_j = sum_{t>=j,h} p_tj dO_th   (response keys only)
//
// One row-stationary kernel serves all three gradients.  A CTA keeps 128 "rows" resident in
// shared memory (operands A1, A2) and streams 64-wide "column" tiles through a ring of
// 16 KB chunks:
//     S = A1 B1^T,  T = A2 B2^T      (tcgen05.mma, operands in shared memory, K-major)
//     E = f(S, T)                     (one thread per row, bf16 written over S in TMEM)
//     ACC += E B3                     (E read from TMEM, B3 MN-major from shared memory)
//   mode DQ: rows = 128 queries of one head, columns = keys of one partial (prefix shard
//            through the page table, or the causal response block); A1 = Q, A2 = dO,
//            B1 = B3 = K, B2 = V; E = p (T - Delta_row).  The prefix needs no dK/dV, so this
//            three-GEMM form is all the prefix ever costs.
//   mode DK: rows = 128 response keys, columns = queries (t >= j) of every head of the group;
//            A1 = K_resp, A2 = V_resp, B1 = B3 = Q, B2 = dO; E = p (T - Delta_col).
//   mode DV: as DK without T; B3 = dO; E = p.
// TMEM columns: ACC [0, D), then two buffers of (S 64 | T 64).
#include <cuda_bf16.h>

#include <mutex>

#include "ls_internal.h"
#include "ls_sm100.cuh"

namespace ls {

enum { MODE_DQ = 0, MODE_DK = 1, MODE_DV = 2 };

struct BwdParams {
  CUtensorMap a1_map, a2_map;                 // stationary rows: box 64 x 128 tokens x 1 group
  // streamed 64-column chunks, box 64 x 64 tokens x D/64 groups
  CUtensorMap bk_map, bk_tail, bv_map, bv_tail;   // prefix pool K and V (mode DQ)
  CUtensorMap b1r_map, b2r_map, b3r_map;          // dense sources: response K/V/K (DQ) or Q/dO/(Q|dO) (DK, DV)
  const int32_t* shard_phys_pages;
  const int32_t* shard_page_offset;
  const int32_t* shard_tail_slot;
  const int64_t* shard_tokens;
  const float* lse;      // [R, Hq]
  const float* delta;    // [R, Hq]
  float* dq_part;        // [(S+1), R, Hq, D] fp32, unscaled (mode DQ)
  __nv_bfloat16* out;    // dk_resp or dv_resp [R, Hkv, D] (modes DK, DV)
  int32_t* status;
  int R, Hq, Hkv, g, S, pg_shift, tiles_per_head, nq_tiles, num_phys_pages;
  float scale, scale_log2;
};

constexpr int kBwdThreads = 192;
constexpr float kLog2e = 1.4426950408889634f;

template <int D>
struct BwdCfg {
  static constexpr int SLABS = D / 64;            // 64-channel groups
  static constexpr int CHUNK = 64 * D * 2;        // one streamed chunk: 64 columns x D channels
  static constexpr int RING = (D == 128) ? 8 : 3;
  static constexpr int A_BYTES = 2 * SLABS * 16384;
  static constexpr int SMEM_BYTES = 1024 + A_BYTES + RING * CHUNK + 512;
};

template <int D, int MODE>
__global__ void __launch_bounds__(kBwdThreads, 1) bwd_kernel(const __grid_constant__ BwdParams p) {
  using C = BwdCfg<D>;
  constexpr bool HAS_T = (MODE != MODE_DV);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* a1_smem = smem;
  uint8_t* a2_smem = smem + C::SLABS * 16384;
  uint8_t* ring = smem + C::A_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + C::RING * C::CHUNK);
  uint64_t* a_full = bars;
  uint64_t* full = bars + 1;
  uint64_t* empty = full + C::RING;
  uint64_t* st_full = empty + C::RING;   // [2] S (and T) of a tile are in TMEM
  uint64_t* e_full = st_full + 2;        // [2] E of a tile is in TMEM
  uint64_t* acc_final = e_full + 2;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_final + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- work item
  int part = 0, kvh, h = 0, row0;          // row0: first query (DQ) or first key (DK, DV) of the tile
  bool is_resp = true;
  int64_t tokens = 0;
  int page_off = 0, n_pages = 0, tail_slot = -1;
  int n_tiles;
  int tt_min = 0, n_tt = 0;                // DK/DV: first 64-query tile and tiles per head
  if (MODE == MODE_DQ) {
    int idx = blockIdx.x;
    const int qtile = idx % p.nq_tiles;
    idx /= p.nq_tiles;
    part = idx % (p.S + 1);
    kvh = idx / (p.S + 1);
    h = kvh * p.g + qtile / p.tiles_per_head;
    row0 = (qtile % p.tiles_per_head) * 128;
    is_resp = (part == p.S);
    if (is_resp) {
      tokens = min(p.R, row0 + 128);
    } else {
      tokens = p.shard_tokens[part];
      page_off = p.shard_page_offset[part];
      n_pages = p.shard_page_offset[part + 1] - page_off;
      tail_slot = p.shard_tail_slot[part];
    }
    n_tiles = (int)((tokens + 63) / 64);
  } else {
    kvh = blockIdx.x / p.tiles_per_head;
    row0 = (blockIdx.x % p.tiles_per_head) * 128;
    tt_min = row0 / 64;
    n_tt = (p.R + 63) / 64 - tt_min;
    n_tiles = p.g * n_tt;
  }

  if (threadIdx.x == 0) {
    mbar_init(a_full, 1);
    for (int i = 0; i < C::RING; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    mbar_init(&st_full[0], 1);
    mbar_init(&st_full[1], 1);
    mbar_init(&e_full[0], 128);
    mbar_init(&e_full[1], 128);
    mbar_init(acc_final, 1);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_holder, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  const uint32_t tmem_acc = tmem_base;
  const uint32_t tmem_buf0 = tmem_base + D;

  if (warp == 0) {
    // =========================================================== producer (one thread)
    if (lane == 0 && n_tiles > 0) {
      mbar_arrive_expect_tx(a_full, (HAS_T ? 2 : 1) * C::SLABS * 16384);
      const int a_head = (MODE == MODE_DQ) ? h : kvh;
      for (int c = 0; c < C::SLABS; ++c) {
        tma_load_5d(a1_smem + c * 16384, &p.a1_map, a_full, 0, row0, c, a_head, 0);
        if (HAS_T) tma_load_5d(a2_smem + c * 16384, &p.a2_map, a_full, 0, row0, c, a_head, 0);
      }
      const int32_t* pages = p.shard_phys_pages + page_off;
      const int pg_mask = (1 << p.pg_shift) - 1;
      const bool dense = (MODE != MODE_DQ) || is_resp;
      auto fetch = [&](int tile) -> int {     // physical page of column tile `tile` (prefix shards only)
        const int ps = (tile * 64) >> p.pg_shift;
        return (!dense && tile < n_tiles && ps < n_pages) ? __ldg(pages + ps) : 0;
      };
      uint32_t slot = 0, phase = 0, issued = 0;
      bool ok = true;
      // one chunk: 64 columns x D channels of source `which` (0: B1, 1: B2, 2: B3) of column tile i
      auto load = [&](int which, int i, int page) {
        ok = ok && mbar_wait(&empty[slot], phase ^ 1, abort_flag);
        if (ok) {
          mbar_arrive_expect_tx(&full[slot], C::CHUNK);
          uint8_t* dst = ring + slot * C::CHUNK;
          if (MODE == MODE_DQ) {
            const int tok = i * 64;
            if (is_resp) {
              tma_load_5d(dst, which == 1 ? &p.b2r_map : &p.b1r_map, &full[slot], 0, tok, 0, kvh, 0);
            } else {
              const bool tail = (tok >> p.pg_shift) == tail_slot;
              const CUtensorMap* m = which == 1 ? (tail ? &p.bv_tail : &p.bv_map) : (tail ? &p.bk_tail : &p.bk_map);
              tma_load_5d(dst, m, &full[slot], 0, tok & pg_mask, 0, kvh, page);
            }
          } else {
            const int hh = kvh * p.g + i / n_tt;
            const int tq = (tt_min + i % n_tt) * 64;
            const CUtensorMap* m = which == 0 ? &p.b1r_map : which == 1 ? &p.b2r_map : &p.b3r_map;
            tma_load_5d(dst, m, &full[slot], 0, tq, 0, hh, 0);
          }
        }
        ++issued;
        if (++slot == (uint32_t)C::RING) { slot = 0; phase ^= 1; }
      };
      // chunk order = consumption order: ST(0) ST(1) [M(i) ST(i+2)] ...
      int pg0 = fetch(0), pg1 = fetch(1), pg2 = fetch(2);      // pages of tiles i, i+1, i+2
      load(0, 0, pg0);
      if (HAS_T) load(1, 0, pg0);
      if (n_tiles > 1) {
        load(0, 1, pg1);
        if (HAS_T) load(1, 1, pg1);
      }
      for (int i = 0; i < n_tiles; ++i) {
        const int pg3 = fetch(i + 3);                          // used two iterations from now
        load(2, i, pg0);
        if (i + 2 < n_tiles) {
          load(0, i + 2, pg2);
          if (HAS_T) load(1, i + 2, pg2);
        }
        pg0 = pg1; pg1 = pg2; pg2 = pg3;
      }
      if (*abort_flag) {   // aborted: wait (bounded) for the copies already started
        for (uint32_t s = 0; s < (uint32_t)C::RING && s < issued; ++s) {
          const uint32_t last = ((issued - 1 - s) / C::RING) * C::RING + s;
          const uint64_t t_start = globaltimer_ns();
          while (!mbar_try_wait(&full[s], (last / C::RING) & 1, 1000) && globaltimer_ns() - t_start < 100000000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // =========================================================== MMA issuer (one thread)
    if (lane == 0 && n_tiles > 0) {
      constexpr uint32_t idesc_st = make_idesc(128, 64, 0, 0);
      constexpr uint32_t idesc_acc = make_idesc(128, D, 0, 1);
      constexpr uint32_t hi = sdesc_hi(1024);
      const uint32_t a1_lo = sdesc_lo(smem_u32(a1_smem), 16), a2_lo = sdesc_lo(smem_u32(a2_smem), 16);
      const uint32_t ring_k_lo = sdesc_lo(smem_u32(ring), 16);      // K-major view of a chunk
      const uint32_t ring_m_lo = sdesc_lo(smem_u32(ring), 8192);    // MN-major view: 8 KB group pitch
      uint32_t slot = 0, phase = 0;
      bool ok = mbar_wait(a_full, 0, abort_flag);
      auto advance = [&]() {
        if (++slot == (uint32_t)C::RING) { slot = 0; phase ^= 1; }
      };
      auto issue_st = [&](int i) {
        const uint32_t buf = tmem_buf0 + (i & 1) * 128;
#pragma unroll
        for (int op = 0; op < (HAS_T ? 2 : 1); ++op) {
          ok = ok && mbar_wait(&full[slot], phase, abort_flag);
          if (!ok) return;
          tc_fence_after();
          const uint32_t a_lo = op == 0 ? a1_lo : a2_lo;
          const uint32_t b_lo = ring_k_lo + slot * (C::CHUNK >> 4);
#pragma unroll
          for (int s = 0; s < C::SLABS; ++s)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              mma_ss(buf + op * 64, sdesc(a_lo + ((s * 16384 + k * 32) >> 4), hi),
                     sdesc(b_lo + ((s * 8192 + k * 32) >> 4), hi), idesc_st, (s | k) != 0);
          mma_commit(&empty[slot]);
          advance();
        }
        mma_commit(&st_full[i & 1]);
      };
      auto issue_acc = [&](int i) {
        const uint32_t e_base = tmem_buf0 + (i & 1) * 128;
        ok = ok && mbar_wait(&full[slot], phase, abort_flag);
        if (!ok) return;
        tc_fence_after();
        const uint32_t b_lo = ring_m_lo + slot * (C::CHUNK >> 4);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          mma_ts(tmem_acc, e_base + kk * 8, sdesc(b_lo + ((kk * 2048) >> 4), hi), idesc_acc, (i | kk) != 0);
        mma_commit(&empty[slot]);
        advance();
        if (i == n_tiles - 1) mma_commit(acc_final);
      };
      if (ok) issue_st(0);
      if (ok && n_tiles > 1) issue_st(1);
      for (int i = 0; i < n_tiles && ok; ++i) {
        ok = ok && mbar_wait(&e_full[i & 1], (i >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        issue_acc(i);
        if (ok && i + 2 < n_tiles) issue_st(i + 2);
      }
    }
  } else {
    // =========================================================== elementwise + epilogue
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int r_idx = row0 + row;                 // query t (DQ) or key j (DK, DV)
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    const bool row_ok = r_idx < p.R;
    float* dq_dst = nullptr;
    if (MODE == MODE_DQ) dq_dst = p.dq_part + (((size_t)part * p.R + min(r_idx, p.R - 1)) * p.Hq + h) * D;
    if (n_tiles == 0) {
      if (MODE == MODE_DQ && row_ok)
        for (int c = 0; c < D; c += 4) *reinterpret_cast<float4*>(dq_dst + c) = make_float4(0.f, 0.f, 0.f, 0.f);
    } else {
      float lse2_row = 0.f, delta_row = 0.f;
      int64_t lim = 0;
      if (MODE == MODE_DQ) {
        const size_t ri = (size_t)min(r_idx, p.R - 1) * p.Hq + h;
        lse2_row = p.lse[ri] * kLog2e;
        delta_row = p.delta[ri];
        lim = is_resp ? (int64_t)min(r_idx, p.R - 1) : tokens - 1;
      }
      bool ok = true;
      for (int i = 0; i < n_tiles && ok; ++i) {
        const uint32_t tb = tmem_buf0 + (i & 1) * 128 + lane_sel;
        // per-column constants (DK, DV): lane L holds columns L and L + 32
        float cl0 = 0.f, cl1 = 0.f, cd0 = 0.f, cd1 = 0.f;
        int tq0 = 0;
        if (MODE != MODE_DQ) {
          const int hh = kvh * p.g + i / n_tt;
          tq0 = (tt_min + i % n_tt) * 64;
          const int ta = min(tq0 + lane, p.R - 1), tb2 = min(tq0 + lane + 32, p.R - 1);
          cl0 = __ldg(p.lse + (size_t)ta * p.Hq + hh) * kLog2e;
          cl1 = __ldg(p.lse + (size_t)tb2 * p.Hq + hh) * kLog2e;
          if (MODE == MODE_DK) {
            cd0 = __ldg(p.delta + (size_t)ta * p.Hq + hh);
            cd1 = __ldg(p.delta + (size_t)tb2 * p.Hq + hh);
          }
        }
        ok = mbar_wait(&st_full[i & 1], (i >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        uint32_t sr[64], tr[64];
        tmem_ld32(tb, sr);
        tmem_ld32(tb + 32, sr + 32);
        if (HAS_T) {
          tmem_ld32(tb + 64, tr);
          tmem_ld32(tb + 96, tr + 32);
        }
        tc_wait_ld32(sr);
        tc_wait_ld32(sr + 32);
        if (HAS_T) {
          tc_wait_ld32(tr);
          tc_wait_ld32(tr + 32);
        }
        uint32_t pk[32];
        if (MODE == MODE_DQ) {
          const int key0 = i * 64;
          const bool edge = __any_sync(0xffffffffu, (int64_t)key0 + 63 > lim);
#pragma unroll
          for (int j = 0; j < 64; j += 2) {
            float p0 = ex2(fmaf(__uint_as_float(sr[j]), p.scale_log2, -lse2_row));
            float p1 = ex2(fmaf(__uint_as_float(sr[j + 1]), p.scale_log2, -lse2_row));
            if (edge) {
              if ((int64_t)key0 + j > lim) p0 = 0.f;
              if ((int64_t)key0 + j + 1 > lim) p1 = 0.f;
            }
            pk[j >> 1] = pack_bf16(p0 * (__uint_as_float(tr[j]) - delta_row),
                                   p1 * (__uint_as_float(tr[j + 1]) - delta_row));
          }
        } else {
          // column t is visible to key row j when j <= t < R
          const bool edge = (tq0 < row0 + 127) || (tq0 + 63 >= p.R);
#pragma unroll
          for (int j = 0; j < 64; j += 2) {
            const float l0 = __shfl_sync(0xffffffffu, (j < 32) ? cl0 : cl1, j & 31);
            const float l1 = __shfl_sync(0xffffffffu, (j + 1 < 32) ? cl0 : cl1, (j + 1) & 31);
            float p0 = ex2(fmaf(__uint_as_float(sr[j]), p.scale_log2, -l0));
            float p1 = ex2(fmaf(__uint_as_float(sr[j + 1]), p.scale_log2, -l1));
            if (edge) {
              const int ta = tq0 + j;
              if (ta < r_idx || ta >= p.R) p0 = 0.f;
              if (ta + 1 < r_idx || ta + 1 >= p.R) p1 = 0.f;
            }
            if (MODE == MODE_DK) {
              const float d0 = __shfl_sync(0xffffffffu, (j < 32) ? cd0 : cd1, j & 31);
              const float d1 = __shfl_sync(0xffffffffu, (j + 1 < 32) ? cd0 : cd1, (j + 1) & 31);
              p0 *= __uint_as_float(tr[j]) - d0;
              p1 *= __uint_as_float(tr[j + 1]) - d1;
            }
            pk[j >> 1] = pack_bf16(p0, p1);
          }
        }
        tmem_st32(tb, pk);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(&e_full[i & 1]);
      }
      if (ok) ok = mbar_wait(acc_final, 0, abort_flag);
      if (ok) {
        tc_fence_after();
        const float out_scale = (MODE == MODE_DK) ? p.scale : 1.0f;
#pragma unroll 1
        for (int c = 0; c < D; c += 32) {
          uint32_t o[32];
          tmem_ld32(tmem_acc + lane_sel + c, o);
          tc_wait_ld32(o);
          if (row_ok) {
            if (MODE == MODE_DQ) {
#pragma unroll
              for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<float4*>(dq_dst + c + j) =
                    make_float4(__uint_as_float(o[j]), __uint_as_float(o[j + 1]), __uint_as_float(o[j + 2]),
                                __uint_as_float(o[j + 3]));
            } else {
              __nv_bfloat16* dst = p.out + ((size_t)r_idx * p.Hkv + kvh) * D + c;
#pragma unroll
              for (int j = 0; j < 32; j += 8) {
                uint4 v;
                v.x = pack_bf16(__uint_as_float(o[j]) * out_scale, __uint_as_float(o[j + 1]) * out_scale);
                v.y = pack_bf16(__uint_as_float(o[j + 2]) * out_scale, __uint_as_float(o[j + 3]) * out_scale);
                v.z = pack_bf16(__uint_as_float(o[j + 4]) * out_scale, __uint_as_float(o[j + 5]) * out_scale);
                v.w = pack_bf16(__uint_as_float(o[j + 6]) * out_scale, __uint_as_float(o[j + 7]) * out_scale);
                *reinterpret_cast<uint4*>(dst + j) = v;
              }
            }
          }
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

// Delta[t,h] = sum_d dO[t,h,d] * O[t,h,d], one warp per row.
__global__ void delta_kernel(const __nv_bfloat16* __restrict__ d_o, const float* __restrict__ o, int64_t rows,
                             int dv, float* __restrict__ delta) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  float acc = 0.f;
  for (int c = lane * 4; c < dv; c += 128) {
    const float4 ov = *reinterpret_cast<const float4*>(o + row * dv + c);
    const uint2 raw = *reinterpret_cast<const uint2*>(d_o + row * dv + c);
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
    acc = fmaf(__low2float(a), ov.x, acc);
    acc = fmaf(__high2float(a), ov.y, acc);
    acc = fmaf(__low2float(b), ov.z, acc);
    acc = fmaf(__high2float(b), ov.w, acc);
  }
  for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
  if (lane == 0) delta[row] = acc;
}

// dQ = scale * sum over partials (Eq. qwen-dq-reduce), fp32 in, bf16 out; fixed summation order.
__global__ void dq_reduce_kernel(const float* __restrict__ dq_part, int parts, int64_t n4, float scale,
                                 __nv_bfloat16* __restrict__ dq) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int r = 0; r < parts; ++r) {
      const float4 v = *reinterpret_cast<const float4*>(dq_part + ((int64_t)r * n4 + i) * 4);
      acc.x += v.x;
      acc.y += v.y;
      acc.z += v.z;
      acc.w += v.w;
    }
    uint2 pk;
    pk.x = pack_bf16(acc.x * scale, acc.y * scale);
    pk.y = pack_bf16(acc.z * scale, acc.w * scale);
    *reinterpret_cast<uint2*>(dq + i * 4) = pk;
  }
}

template <int D, int MODE>
static ls_status_t launch_bwd(const BwdParams& prm, int grid, cudaStream_t st) {
  using C = BwdCfg<D>;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(bwd_kernel<D, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) !=
        cudaSuccess)
      return LS_ERR_CUDA;
    configured = true;
  }
  constexpr int which = MODE == MODE_DQ ? LS_KERNEL_BWD_DQ : MODE == MODE_DK ? LS_KERNEL_BWD_DK : LS_KERNEL_BWD_DV;
  profile_begin(which, st);
  bwd_kernel<D, MODE><<<grid, kBwdThreads, C::SMEM_BYTES, st>>>(prm);
  profile_end(which, st);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

}  // namespace ls

extern "C" ls_status_t ls_replay_attn_bwd(const ls_pages_t* h, const ls_attn_params_t* prm, const void* q,
                                          const void* k_resp, const void* v_resp, const float* o_f32,
                                          const float* lse, const void* d_o, void* dq, void* dk_resp,
                                          void* dv_resp, void* workspace, size_t workspace_bytes,
                                          int32_t* status_dev, void* stream) {
  if (!h || !prm || !q || !k_resp || !v_resp || !o_f32 || !lse || !d_o || !dq || !dk_resp || !dv_resp)
    return LS_ERR_INVALID_ARG;
  if (!h->on_device) return LS_ERR_INVALID_ARG;
  const ls_pages_desc_t& d = h->desc;
  if (prm->R < 1 || prm->num_q_heads < 1 || prm->num_q_heads % d.num_kv_heads != 0) return LS_ERR_INVALID_ARG;
  if (!(prm->scale > 0.f)) return LS_ERR_INVALID_ARG;
  const bool mla = d.dim_k == 576 && d.dim_v == 512;
  if (!((d.dim_k == 128 && d.dim_v == 128) || (d.dim_k == 256 && d.dim_v == 256) || mla))
    return LS_ERR_UNSUPPORTED_SHAPE;
  const void* ptrs[] = {q, k_resp, v_resp, o_f32, d_o, dq, dk_resp, dv_resp, workspace};
  for (const void* ptr : ptrs)
    if (!ls::aligned16(ptr)) return LS_ERR_ALIGNMENT;
  const size_t need = ls_replay_attn_workspace_bytes(h, prm, LS_WORKSPACE_BWD);
  if (!workspace || workspace_bytes < need) return LS_ERR_WORKSPACE;

  const int R = prm->R, Hq = prm->num_q_heads, Hkv = d.num_kv_heads, D = d.dim_k;
  const int64_t rows = (int64_t)R * Hq;
  float* dq_part = static_cast<float*>(workspace);
  float* delta = dq_part + (size_t)(d.num_shards + 1) * rows * D;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);

  ls::delta_kernel<<<(int)((rows + 7) / 8), 256, 0, cs>>>(static_cast<const __nv_bfloat16*>(d_o), o_f32, rows,
                                                        d.dim_v, delta);

  if (mla) {
    ls_status_t ms = ls::bwd_mla(h, prm, q, k_resp, v_resp, lse, delta, d_o, dq_part, dk_resp, dv_resp, status_dev, cs);
    if (ms != LS_OK) return ms;
    const int64_t n4m = rows * D / 4;
    ls::dq_reduce_kernel<<<(int)std::min<int64_t>((n4m + 255) / 256, 148 * 16), 256, 0, cs>>>(
        dq_part, d.num_shards + 1, n4m, prm->scale, static_cast<__nv_bfloat16*>(dq));
    return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
  }

  auto dense_map = [&](CUtensorMap* m, const void* base, int heads, int box_tok, int groups) {
    return ls::encode_map5(m, base, D, R, heads, 1, (int64_t)heads * D, D, (int64_t)R * heads * D, box_tok, groups);
  };
  const int groups = D / 64;
  ls::BwdParams P;
  P.shard_phys_pages = h->d_shard_phys_pages;
  P.shard_page_offset = h->d_shard_page_offset;
  P.shard_tail_slot = h->d_shard_tail_slot;
  P.shard_tokens = h->d_shard_tokens;
  P.lse = lse;
  P.delta = delta;
  P.dq_part = dq_part;
  P.out = nullptr;
  P.status = status_dev;
  P.R = R;
  P.Hq = Hq;
  P.Hkv = Hkv;
  P.g = Hq / Hkv;
  P.S = d.num_shards;
  P.pg_shift = d.page_size == 64 ? 6 : d.page_size == 128 ? 7 : d.page_size == 256 ? 8 : 9;
  P.tiles_per_head = (R + 127) / 128;
  P.nq_tiles = P.g * P.tiles_per_head;
  P.num_phys_pages = (int)std::min<int64_t>(d.num_phys_pages, INT32_MAX);
  P.scale = prm->scale;
  P.scale_log2 = prm->scale * ls::kLog2e;

  // ---- dQ: rows = queries, columns = keys of every partial
  ls_status_t st = dense_map(&P.a1_map, q, Hq, 128, 1);
  if (st == LS_OK) st = dense_map(&P.a2_map, d_o, Hq, 128, 1);
  if (st == LS_OK) st = dense_map(&P.b1r_map, k_resp, Hkv, 64, groups);
  if (st == LS_OK) st = dense_map(&P.b2r_map, v_resp, Hkv, 64, groups);
  if (st == LS_OK) st = ls::encode_pool_map5(&P.bk_map, h, 0, 64, groups, false);
  if (st == LS_OK) st = ls::encode_pool_map5(&P.bk_tail, h, 0, 64, groups, true);
  if (st == LS_OK) st = ls::encode_pool_map5(&P.bv_map, h, 1, 64, groups, false);
  if (st == LS_OK) st = ls::encode_pool_map5(&P.bv_tail, h, 1, 64, groups, true);
  if (st != LS_OK) return st;
  P.b3r_map = P.b1r_map;
  const int64_t grid_dq = (int64_t)Hkv * (d.num_shards + 1) * P.nq_tiles;
  if (grid_dq > INT32_MAX) return LS_ERR_UNSUPPORTED_SHAPE;
  st = (D == 128) ? ls::launch_bwd<128, ls::MODE_DQ>(P, (int)grid_dq, cs)
                  : ls::launch_bwd<256, ls::MODE_DQ>(P, (int)grid_dq, cs);
  if (st != LS_OK) return st;
  const int64_t n4 = rows * D / 4;
  ls::dq_reduce_kernel<<<(int)std::min<int64_t>((n4 + 255) / 256, 148 * 16), 256, 0, cs>>>(
      dq_part, d.num_shards + 1, n4, prm->scale, static_cast<__nv_bfloat16*>(dq));

  // ---- dK and dV of the response keys: rows = keys, columns = queries of the KV group
  const int grid_kv = Hkv * P.tiles_per_head;
  st = dense_map(&P.a1_map, k_resp, Hkv, 128, 1);
  if (st == LS_OK) st = dense_map(&P.a2_map, v_resp, Hkv, 128, 1);
  if (st == LS_OK) st = dense_map(&P.b1r_map, q, Hq, 64, groups);
  if (st == LS_OK) st = dense_map(&P.b2r_map, d_o, Hq, 64, groups);
  if (st != LS_OK) return st;
  P.b3r_map = P.b1r_map;
  P.out = static_cast<__nv_bfloat16*>(dk_resp);
  st = (D == 128) ? ls::launch_bwd<128, ls::MODE_DK>(P, grid_kv, cs) : ls::launch_bwd<256, ls::MODE_DK>(P, grid_kv, cs);
  if (st != LS_OK) return st;
  P.b3r_map = P.b2r_map;
  P.out = static_cast<__nv_bfloat16*>(dv_resp);
  st = (D == 128) ? ls::launch_bwd<128, ls::MODE_DV>(P, grid_kv, cs) : ls::launch_bwd<256, ls::MODE_DV>(P, grid_kv, cs);
  if (st != LS_OK) return st;
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

// ---------------------------------------------------------------------------------
// Backward without caller scratch: the per-partial dQ sums and Delta live in a fixed
// array inside the library's device image instead of a caller-provided workspace.
// ---------------------------------------------------------------------------------
namespace ls {

constexpr size_t kStaticScratchBytes = LS_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_bwd_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static void* g_scratch_ptr[kMaxDevices] = {};
static std::mutex g_scratch_mutex;

// Device address of g_bwd_scratch on the current device.  In host code the array's name is
// only a handle for the runtime, never an address a kernel could use, so the address is
// looked up once per device (with that device current) and cached.
static ls_status_t static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LS_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_bwd_scratch) != cudaSuccess || !ptr) return LS_ERR_CUDA;
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return LS_OK;
}

}  // namespace ls

extern "C" size_t ls_replay_attn_bwd_static_capacity(void) { return ls::kStaticScratchBytes; }

extern "C" ls_status_t ls_replay_attn_bwd_static(const ls_pages_t* h, const ls_attn_params_t* prm, const void* q,
                                                 const void* k_resp, const void* v_resp, const float* o_f32,
                                                 const float* lse, const void* d_o, void* dq, void* dk_resp,
                                                 void* dv_resp, int32_t* status_dev, void* stream) {
  if (!h || !prm) return LS_ERR_INVALID_ARG;
  const size_t need = ls_replay_attn_workspace_bytes(h, prm, LS_WORKSPACE_BWD);
  if (need == 0) return LS_ERR_INVALID_ARG;
  if (need > ls::kStaticScratchBytes) return LS_ERR_WORKSPACE;   // shape too large for the built-in scratch
  void* scratch = nullptr;
  ls_status_t st = ls::static_scratch(&scratch);
  if (st != LS_OK) return st;
  // Nothing in the scratch has to start at zero: the dQ pass writes every partial of every
  // row (zeros for an empty partial) and the Delta kernel writes every row before either
  // is read, so the previous call's leftovers are never observed.
  return ls_replay_attn_bwd(h, prm, q, k_resp, v_resp, o_f32, lse, d_o, dq, dk_resp, dv_resp, scratch,
                            ls::kStaticScratchBytes, status_dev, stream);
}
