// Replay backward for the shared-latent shape: key page of 576 channels (512 latent + 64
// rope) whose first 512 channels are also the value (Sec. "GLM page payloads"; the dense
// form of that attention).  Same mathematics as ls_bwd.cu:
//   ds = p (dO . v - Delta);  dQ = scale * ds K;  dK_resp = scale * ds^T Q;  dV_resp = p^T dO.
//
// What differs is the budget.  Q (576) and dO (512) of 128 rows do not fit in shared memory
// together, and a 576-column fp32 accumulator does not fit in TMEM beside the score buffers.
// So a CTA keeps 64 rows resident (the tensor-core instructions still span 128 rows; the
// upper 64 compute on whatever bytes follow and are never read back) and covers the
// accumulator in passes of NACC 64-channel groups, recomputing S and T in every pass.
// Everything is streamed in 8 KB slabs of 64 columns x 64 channels.
//
//   mode DQ: rows = 64 queries of one head; columns = keys of one partial;
//            S = Q K^T (9 slabs), T = dO V^T (8 slabs), E = p (T - Delta_row),
//            ACC[:, pass] += E K[:, pass]                      (3 passes x 192 channels)
//   mode DK: rows = 64 response keys; columns = queries t >= j of every head;
//            S = K Q^T, T = V dO^T, E = p (T - Delta_col), ACC += E Q   (3 x 192)
//   mode DV: S only, E = p, ACC += E dO                        (2 passes x 256 channels)
// TMEM columns: ACC [0, 64 NACC), then two buffers of (S 64 | T 64) from column 256.
#include <cuda_bf16.h>

#include <algorithm>

#include "ls_internal.h"
#include "ls_sm100.cuh"

namespace ls {

enum { MLA_DQ = 0, MLA_DK = 1, MLA_DV = 2 };

struct MlaBwdParams {
  CUtensorMap a1_map, a2_map;        // resident rows: box 64 ch x 64 tokens
  CUtensorMap bk_map, bk_tail;       // prefix pool key page, box 64 x 64 (mode DQ)
  CUtensorMap bv_map, bv_tail;       // prefix pool values (the key page again when aliased)
  CUtensorMap b1r_map, b2r_map, b3r_map;   // dense sources: response K/V/K (DQ) or Q/dO/(Q|dO)
  const int32_t* shard_phys_pages;
  const int32_t* shard_page_offset;
  const int32_t* shard_tail_slot;
  const int64_t* shard_tokens;
  const float* lse;
  const float* delta;
  float* dq_part;          // [(S+1), R, Hq, 576] fp32, unscaled
  __nv_bfloat16* out;      // dk_resp [R, Hkv, 576] or dv_resp [R, Hkv, 512]
  int32_t* status;
  int R, Hq, Hkv, g, S, pg_shift, tiles_per_head, nq_tiles, num_phys_pages;   // tiles of 64 rows
  int part_first, part_count;   // mode DQ: partials [part_first, part_first + part_count) are computed
  // modes DK / DV: the heads of a KV group are cut into hsplit ranges, one CTA each per key tile and
  // pass (a short response has too few key tiles to fill the GPU); with more than one the fp32 sums
  // go to kv_part [hsplit, R, Hkv, 576 | 512] and a reduce kernel writes `out`
  int hsplit;
  float* kv_part;
  float scale, scale_log2;
};

constexpr int kMlaThreads = 192;
constexpr int kSlab = 8192;             // 64 rows x 128 B
constexpr int kD1 = 576, kD2 = 512;
constexpr int kS1 = kD1 / 64, kS2 = kD2 / 64;
constexpr int kMlaRing = 10;
constexpr int kMlaSmem = 1024 + (kS1 + kS2 + kMlaRing) * kSlab + 512;
constexpr float kLog2eMla = 1.4426950408889634f;

template <int MODE>
__global__ void __launch_bounds__(kMlaThreads, 1) bwd_mla_kernel(const __grid_constant__ MlaBwdParams p) {
  constexpr bool HAS_T = (MODE != MLA_DV);
  constexpr int NACC = (MODE == MLA_DV) ? 4 : 3;              // 64-channel groups per pass
  constexpr int NPASS = (MODE == MLA_DV) ? kS2 / 4 : kS1 / 3;
  constexpr int OUT_D = (MODE == MLA_DV) ? kD2 : kD1;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* a1_smem = smem;
  uint8_t* a2_smem = smem + kS1 * kSlab;
  uint8_t* ring = a2_smem + kS2 * kSlab;
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + kMlaRing * kSlab);
  uint64_t* a_full = bars;
  uint64_t* full = bars + 1;
  uint64_t* empty = full + kMlaRing;
  uint64_t* st_full = empty + kMlaRing;   // [2]
  uint64_t* e_full = st_full + 2;         // [2]
  uint64_t* acc_final = e_full + 2;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_final + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- work item (pass is the fastest index: the passes of one tile share their loads in L2)
  int idx = blockIdx.x;
  const int pass = idx % NPASS;
  idx /= NPASS;
  int part = 0, kvh, h = 0, row0, hs = 0, h_lo = 0;
  bool is_resp = true;
  int64_t tokens = 0;
  int page_off = 0, n_pages = 0, tail_slot = -1, n_tiles, tt_min = 0, n_tt = 0;
  if (MODE == MLA_DQ) {
    const int qtile = idx % p.nq_tiles;
    idx /= p.nq_tiles;
    part = p.part_first + idx % p.part_count;
    kvh = idx / p.part_count;
    h = kvh * p.g + qtile / p.tiles_per_head;
    row0 = (qtile % p.tiles_per_head) * 64;
    is_resp = (part == p.S);
    if (is_resp) {
      tokens = min(p.R, row0 + 64);
    } else {
      tokens = p.shard_tokens[part];
      page_off = p.shard_page_offset[part];
      n_pages = p.shard_page_offset[part + 1] - page_off;
      tail_slot = p.shard_tail_slot[part];
    }
    n_tiles = (int)((tokens + 63) / 64);
  } else {
    hs = idx % p.hsplit;
    idx /= p.hsplit;
    kvh = idx / p.tiles_per_head;
    row0 = (idx % p.tiles_per_head) * 64;
    tt_min = row0 / 64;
    n_tt = (p.R + 63) / 64 - tt_min;
    h_lo = (int)((long long)hs * p.g / p.hsplit);
    n_tiles = ((int)((long long)(hs + 1) * p.g / p.hsplit) - h_lo) * n_tt;
  }

  if (threadIdx.x == 0) {
    mbar_init(a_full, 1);
    for (int i = 0; i < kMlaRing; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    mbar_init(&st_full[0], 1);
    mbar_init(&st_full[1], 1);
    mbar_init(&e_full[0], 64);
    mbar_init(&e_full[1], 64);
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
  const uint32_t tmem_buf0 = tmem_base + 256;

  if (warp == 0) {
    // =========================================================== producer (one thread)
    if (lane == 0 && n_tiles > 0) {
      mbar_arrive_expect_tx(a_full, (kS1 + (HAS_T ? kS2 : 0)) * kSlab);
      const int a_head = (MODE == MLA_DQ) ? h : kvh;
      for (int c = 0; c < kS1; ++c) tma_load_5d(a1_smem + c * kSlab, &p.a1_map, a_full, 0, row0, c, a_head, 0);
      if (HAS_T)
        for (int c = 0; c < kS2; ++c) tma_load_5d(a2_smem + c * kSlab, &p.a2_map, a_full, 0, row0, c, a_head, 0);

      const int32_t* pages = p.shard_phys_pages + page_off;
      const int pg_mask = (1 << p.pg_shift) - 1;
      const bool dense = (MODE != MLA_DQ) || is_resp;
      auto fetch = [&](int tile) -> int {
        const int ps = (tile * 64) >> p.pg_shift;
        if (dense) return 0;
        return (tile < n_tiles && ps < n_pages) ? __ldg(pages + ps) : p.num_phys_pages;   // past the end: TMA fills zeros
      };
      uint32_t slot = 0, phase = 0, issued = 0;
      bool ok = true;
      // one slab: 64 columns x 64 channels (group c) of source `which` (0: B1, 1: B2, 2: B3) of tile i
      auto load = [&](int which, int i, int c, int page, int hh, int tq) {
        ok = ok && mbar_wait(&empty[slot], phase ^ 1, abort_flag);
        if (ok) {
          mbar_arrive_expect_tx(&full[slot], kSlab);
          uint8_t* dst = ring + slot * kSlab;
          if (MODE == MLA_DQ) {
            const int tok = i * 64;
            if (is_resp) {
              tma_load_5d(dst, which == 1 ? &p.b2r_map : &p.b1r_map, &full[slot], 0, tok, c, kvh, 0);
            } else {
              const bool tail = (tok >> p.pg_shift) == tail_slot;
              const CUtensorMap* m = which == 1 ? (tail ? &p.bv_tail : &p.bv_map) : (tail ? &p.bk_tail : &p.bk_map);
              tma_load_5d(dst, m, &full[slot], 0, tok & pg_mask, c, kvh, page);
            }
          } else {
            const CUtensorMap* m = which == 0 ? &p.b1r_map : which == 1 ? &p.b2r_map : &p.b3r_map;
            tma_load_5d(dst, m, &full[slot], 0, tq, c, hh, 0);
          }
        }
        ++issued;
        if (++slot == (uint32_t)kMlaRing) { slot = 0; phase ^= 1; }
      };
      auto load_st = [&](int i, int page) {
        const int hh = (MODE == MLA_DQ) ? 0 : kvh * p.g + h_lo + i / n_tt;
        const int tq = (MODE == MLA_DQ) ? 0 : (tt_min + i % n_tt) * 64;
        for (int c = 0; c < kS1; ++c) load(0, i, c, page, hh, tq);
        if (HAS_T)
          for (int c = 0; c < kS2; ++c) load(1, i, c, page, hh, tq);
      };
      auto load_m = [&](int i, int page) {
        const int hh = (MODE == MLA_DQ) ? 0 : kvh * p.g + h_lo + i / n_tt;
        const int tq = (MODE == MLA_DQ) ? 0 : (tt_min + i % n_tt) * 64;
        for (int c = 0; c < NACC; ++c) load(2, i, pass * NACC + c, page, hh, tq);
      };
      int pg0 = fetch(0), pg1 = fetch(1), pg2 = fetch(2);
      load_st(0, pg0);
      if (n_tiles > 1) load_st(1, pg1);
      for (int i = 0; i < n_tiles; ++i) {
        const int pg3 = fetch(i + 3);
        load_m(i, pg0);
        if (i + 2 < n_tiles) load_st(i + 2, pg2);
        pg0 = pg1; pg1 = pg2; pg2 = pg3;
      }
      if (*abort_flag) {   // aborted: wait (bounded) for the copies already started
        for (uint32_t s = 0; s < (uint32_t)kMlaRing && s < issued; ++s) {
          const uint32_t last = ((issued - 1 - s) / kMlaRing) * kMlaRing + s;
          const uint64_t t_start = globaltimer_ns();
          while (!mbar_try_wait(&full[s], (last / kMlaRing) & 1, 1000) && globaltimer_ns() - t_start < 100000000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // =========================================================== MMA issuer (one thread)
    if (lane == 0 && n_tiles > 0) {
      constexpr uint32_t idesc_st = make_idesc(128, 64, 0, 0);
      constexpr uint32_t idesc_acc = make_idesc(128, 64, 0, 1);
      constexpr uint32_t hi = sdesc_hi(1024);
      const uint32_t a1_lo = sdesc_lo(smem_u32(a1_smem), 16), a2_lo = sdesc_lo(smem_u32(a2_smem), 16);
      const uint32_t ring_lo = sdesc_lo(smem_u32(ring), 16);
      uint32_t slot = 0, phase = 0;
      bool ok = mbar_wait(a_full, 0, abort_flag);
      auto advance = [&]() {
        if (++slot == (uint32_t)kMlaRing) { slot = 0; phase ^= 1; }
      };
      auto issue_st = [&](int i) {
        const uint32_t buf = tmem_buf0 + (i & 1) * 128;
        for (int op = 0; op < (HAS_T ? 2 : 1); ++op) {
          const uint32_t a_lo = op == 0 ? a1_lo : a2_lo;
          const int nslab = op == 0 ? kS1 : kS2;
          for (int c = 0; c < nslab; ++c) {
            ok = ok && mbar_wait(&full[slot], phase, abort_flag);
            if (!ok) return;
            tc_fence_after();
            const uint32_t b_lo = ring_lo + slot * (kSlab >> 4);
#pragma unroll
            for (int k = 0; k < 4; ++k)
              mma_ss(buf + op * 64, sdesc(a_lo + ((c * kSlab + k * 32) >> 4), hi), sdesc(b_lo + ((k * 32) >> 4), hi),
                     idesc_st, (c | k) != 0);
            mma_commit(&empty[slot]);
            advance();
          }
        }
        mma_commit(&st_full[i & 1]);
      };
      auto issue_acc = [&](int i) {
        const uint32_t e_base = tmem_buf0 + (i & 1) * 128;
        for (int c = 0; c < NACC; ++c) {
          ok = ok && mbar_wait(&full[slot], phase, abort_flag);
          if (!ok) return;
          tc_fence_after();
          const uint32_t b_lo = ring_lo + slot * (kSlab >> 4);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            mma_ts(tmem_acc + c * 64, e_base + kk * 8, sdesc(b_lo + ((kk * 2048) >> 4), hi), idesc_acc,
                   (i | kk) != 0);
          mma_commit(&empty[slot]);
          advance();
        }
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
  } else if ((warp & 3) < 2) {
    // =========================================================== elementwise + epilogue
    // only TMEM lanes 0..63 hold real rows: warps 4 and 5 own them
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int r_idx = row0 + row;
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    const bool row_ok = r_idx < p.R;
    float* dq_dst = nullptr;
    if (MODE == MLA_DQ)
      dq_dst = p.dq_part + (((size_t)(part - p.part_first) * p.R + min(r_idx, p.R - 1)) * p.Hq + h) * kD1 + pass * NACC * 64;
    if (n_tiles == 0) {
      if (MODE == MLA_DQ && row_ok)
        for (int c = 0; c < NACC * 64; c += 4) *reinterpret_cast<float4*>(dq_dst + c) = make_float4(0.f, 0.f, 0.f, 0.f);
    } else {
      float lse2_row = 0.f, delta_row = 0.f;
      int64_t lim = 0;
      if (MODE == MLA_DQ) {
        const size_t ri = (size_t)min(r_idx, p.R - 1) * p.Hq + h;
        lse2_row = p.lse[ri] * kLog2eMla;
        delta_row = p.delta[ri];
        lim = is_resp ? (int64_t)min(r_idx, p.R - 1) : tokens - 1;
      }
      bool ok = true;
      for (int i = 0; i < n_tiles && ok; ++i) {
        const uint32_t tb = tmem_buf0 + (i & 1) * 128 + lane_sel;
        float cl0 = 0.f, cl1 = 0.f, cd0 = 0.f, cd1 = 0.f;
        int tq0 = 0;
        if (MODE != MLA_DQ) {
          const int hh = kvh * p.g + h_lo + i / n_tt;
          tq0 = (tt_min + i % n_tt) * 64;
          const int ta = min(tq0 + lane, p.R - 1), tb2 = min(tq0 + lane + 32, p.R - 1);
          cl0 = __ldg(p.lse + (size_t)ta * p.Hq + hh) * kLog2eMla;
          cl1 = __ldg(p.lse + (size_t)tb2 * p.Hq + hh) * kLog2eMla;
          if (MODE == MLA_DK) {
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
        if (MODE == MLA_DQ) {
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
          const bool edge = (tq0 < row0 + 63) || (tq0 + 63 >= p.R);
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
            if (MODE == MLA_DK) {
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
        const float out_scale = (MODE == MLA_DK) ? p.scale : 1.0f;
#pragma unroll 1
        for (int c = 0; c < NACC * 64; c += 32) {
          uint32_t o[32];
          tmem_ld32(tmem_acc + lane_sel + c, o);
          tc_wait_ld32(o);
          if (row_ok) {
            if (MODE == MLA_DQ) {
#pragma unroll
              for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<float4*>(dq_dst + c + j) =
                    make_float4(__uint_as_float(o[j]), __uint_as_float(o[j + 1]), __uint_as_float(o[j + 2]),
                                __uint_as_float(o[j + 3]));
            } else if (p.hsplit > 1) {
              float* dst = p.kv_part + (((size_t)hs * p.R + r_idx) * p.Hkv + kvh) * OUT_D + pass * NACC * 64 + c;
#pragma unroll
              for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<float4*>(dst + j) =
                    make_float4(__uint_as_float(o[j]) * out_scale, __uint_as_float(o[j + 1]) * out_scale,
                                __uint_as_float(o[j + 2]) * out_scale, __uint_as_float(o[j + 3]) * out_scale);
            } else {
              __nv_bfloat16* dst = p.out + ((size_t)r_idx * p.Hkv + kvh) * OUT_D + pass * NACC * 64 + c;
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

template <int MODE>
static ls_status_t launch_mla(const MlaBwdParams& prm, int64_t grid, cudaStream_t st, bool timed = true) {
  static bool configured[64] = {};
  if (grid > INT32_MAX) return LS_ERR_UNSUPPORTED_SHAPE;
  const ls_status_t cfg = configure_smem(bwd_mla_kernel<MODE>, kMlaSmem, configured);
  if (cfg != LS_OK) return cfg;
  constexpr int which = MODE == MLA_DQ ? LS_KERNEL_BWD_DQ : MODE == MLA_DK ? LS_KERNEL_BWD_DK : LS_KERNEL_BWD_DV;
  if (timed) profile_begin(which, st);
  bwd_mla_kernel<MODE><<<(int)grid, kMlaThreads, kMlaSmem, st>>>(prm);
  if (timed) profile_end(which, st);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

int mla_kv_hsplit(const ls_pages* h, int R, int Hq) {
  const int Hkv = h->desc.num_kv_heads;
  const int64_t ctas = (int64_t)Hkv * ((R + 63) / 64) * 3;       // key tiles x passes of the dK launch
  if (ctas >= 148) return 1;
  return (int)std::max<int64_t>(1, std::min<int64_t>(Hq / Hkv, (2 * 148 + ctas - 1) / ctas));
}

// out = bf16(sum of the head ranges' fp32 sums)
__global__ void mla_kv_reduce_kernel(const float* __restrict__ part, int hsplit, int64_t n4, __nv_bfloat16* __restrict__ out) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < hsplit; ++s) {
      const float4 v = *reinterpret_cast<const float4*>(part + ((int64_t)s * n4 + i) * 4);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    uint2 pk;
    pk.x = pack_bf16(acc.x, acc.y);
    pk.y = pack_bf16(acc.z, acc.w);
    *reinterpret_cast<uint2*>(out + i * 4) = pk;
  }
}

// dq_part (fp32, unscaled; only the response block's partial, at index 0, when dq_resp_only)
// and dk_resp / dv_resp (bf16) of the 576/512 shape.
ls_status_t bwd_mla(const ls_pages* h, const ls_attn_params_t* prm, const void* q, const void* k_resp,
                    const void* v_resp, const float* lse, const float* delta, const void* d_o, float* dq_part,
                    void* dk_resp, void* dv_resp, bool dq_resp_only, float* kv_scratch, int32_t* status_dev,
                    cudaStream_t cs) {
  const ls_pages_desc_t& d = h->desc;
  const int R = prm->R, Hq = prm->num_q_heads, Hkv = d.num_kv_heads;
  auto dense_map = [&](CUtensorMap* m, const void* base, int heads, int dim) {
    return encode_map5(m, base, dim, R, heads, 1, (int64_t)heads * dim, dim, (int64_t)R * heads * dim, 64, 1);
  };
  MlaBwdParams P;
  P.shard_phys_pages = h->d_part_pages;
  P.shard_page_offset = h->d_part_page_offset;
  P.shard_tail_slot = h->d_part_tail_slot;
  P.shard_tokens = h->d_part_tokens;
  P.lse = lse;
  P.delta = delta;
  P.dq_part = dq_part;
  P.out = nullptr;
  P.status = status_dev;
  P.R = R;
  P.Hq = Hq;
  P.Hkv = Hkv;
  P.g = Hq / Hkv;
  P.S = h->num_parts();
  P.pg_shift = pg_shift_of(d.page_size);
  P.tiles_per_head = (R + 63) / 64;
  P.nq_tiles = P.g * P.tiles_per_head;
  P.num_phys_pages = (int)std::min<int64_t>(d.num_phys_pages, INT32_MAX);
  P.part_first = dq_resp_only ? P.S : 0;
  P.part_count = dq_resp_only ? 1 : P.S + 1;
  P.hsplit = kv_scratch ? mla_kv_hsplit(h, R, Hq) : 1;
  P.kv_part = kv_scratch;
  P.scale = prm->scale;
  P.scale_log2 = prm->scale * kLog2eMla;

  ls_status_t st = dense_map(&P.a1_map, q, Hq, kD1);
  if (st == LS_OK) st = dense_map(&P.a2_map, d_o, Hq, kD2);
  if (st == LS_OK) st = dense_map(&P.b1r_map, k_resp, Hkv, kD1);
  if (st == LS_OK) st = dense_map(&P.b2r_map, v_resp, Hkv, kD2);
  if (st == LS_OK) st = pool_map(&P.bk_map, h, 0, 64, 1, false);
  if (st == LS_OK) st = pool_map(&P.bk_tail, h, 0, 64, 1, true);
  if (st == LS_OK) st = pool_map(&P.bv_map, h, 1, 64, 1, false);
  if (st == LS_OK) st = pool_map(&P.bv_tail, h, 1, 64, 1, true);
  if (st != LS_OK) return st;
  P.b3r_map = P.b1r_map;
  st = launch_mla<MLA_DQ>(P, (int64_t)Hkv * P.part_count * P.nq_tiles * 3, cs, !dq_resp_only);
  if (st != LS_OK) return st;

  st = dense_map(&P.a1_map, k_resp, Hkv, kD1);
  if (st == LS_OK) st = dense_map(&P.a2_map, v_resp, Hkv, kD2);
  if (st == LS_OK) st = dense_map(&P.b1r_map, q, Hq, kD1);
  if (st == LS_OK) st = dense_map(&P.b2r_map, d_o, Hq, kD2);
  if (st != LS_OK) return st;
  P.b3r_map = P.b1r_map;
  P.out = static_cast<__nv_bfloat16*>(dk_resp);
  auto reduce = [&](int dim, void* out) -> ls_status_t {
    if (P.hsplit == 1) return LS_OK;
    const int64_t n4 = (int64_t)R * Hkv * dim / 4;
    mla_kv_reduce_kernel<<<(int)std::min<int64_t>((n4 + 255) / 256, 148 * 8), 256, 0, cs>>>(
        kv_scratch, P.hsplit, n4, static_cast<__nv_bfloat16*>(out));
    return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
  };
  st = launch_mla<MLA_DK>(P, (int64_t)Hkv * P.tiles_per_head * P.hsplit * 3, cs);
  if (st == LS_OK) st = reduce(kD1, dk_resp);
  if (st != LS_OK) return st;
  P.b3r_map = P.b2r_map;
  P.out = static_cast<__nv_bfloat16*>(dv_resp);
  st = launch_mla<MLA_DV>(P, (int64_t)Hkv * P.tiles_per_head * P.hsplit * 2, cs);
  if (st == LS_OK) st = reduce(kD2, dv_resp);
  return st;
}

}  // namespace ls
