// Replay backward with a detached prefix (Sec. "Lazy Gradient Pages", Eq. qwen-dq-reduce)
// for sm_100a.
//
//   Delta_th = dO_th . O_th;  p_tj = exp(s_tj - LSE_th);  ds_tj = p_tj (dO_th . v_j - Delta_th)
//   dQ_th = scale * sum_j ds_tj k_j      (prefix, suffix and response keys)
//   dK_j  = scale * sum_{t,h} ds_tj q_th,   dV_j = sum_{t,h} p_tj dO_th   (response and suffix keys only)
//
// All kernels are row-stationary: a CTA keeps 128 "rows" resident in shared memory (operands
// A1, A2) and streams "column" tiles through a small ring of chunks:
//     S = A1 B1^T,  T = A2 B2^T      (tcgen05.mma, operands in shared memory)
//     E = f(S, T)                     (row threads; bf16, written over S in TMEM, quarter by quarter)
//     ACC += E B3                     (E read from TMEM, B3 MN-major from shared memory)
//   dQ pass (bwd_dq3_kernel for head dim 256, bwd_dq2_kernel for 128; CTA pairs): rows = queries
//            of one head, columns = keys of one part (prefix sub-shard or suffix block through
//            the page table, or the causal response block); A1 = Q, A2 = dO, B1 = B3 = K,
//            B2 = V; E = p (T - Delta_row).  The prefix needs no dK/dV, so this three-GEMM form
//            is all the prefix ever costs.  The parts of one row tile are summed in a fixed
//            order through one fp32 running dQ (ordered hand-over between CTAs); the last part
//            writes the scaled bf16 result.
//   dK / dV pass (bwd_kv_kernel): rows = 128 keys -- of the response block (columns = queries
//            t >= j of every head of the group) or of a suffix block read through its pages
//            (columns = every query); A1 = K, A2 = V, B1 = B3 = Q, B2 = dO; E = p (T - Delta_col)
//            for dK, E = p with B3 = dO for dV.
#include <cuda_bf16.h>

#include <mutex>

#include "ls_internal.h"
#include "ls_sm100.cuh"

namespace ls {

enum { MODE_DK = 1, MODE_DV = 2 };

struct BwdParams {
  CUtensorMap a1_map, a2_map;                 // stationary rows: box 64 x 128 tokens x 1 group
  CUtensorMap b1r_map, b2r_map, b3r_map;      // dK / dV pass: Q / dO / (Q | dO) as 128 columns x 128 channels;
                                              // single-CTA dQ pass: response K / V the same way
  // single-CTA dQ pass: pool K and V as chunks of 128 keys x 128 channels (box 64 x 128 tokens x 2 groups,
  // or 64 x 64 x 1 on 64-token pages: four boxes per chunk)
  CUtensorMap bk_map, bk_tail, bv_map, bv_tail;
  // dQ pass on CTA pairs: each CTA loads half of every streamed operand.
  //   *_s: 64 columns x 128 channels (box 64 x 64 tokens x 2 groups)
  //   *_m: 128 columns x 64 channels (box 64 x 128 x 1, or 64 x 64 x 1 on 64-token pages)
  CUtensorMap pk_s, pk_s_tail, pv_s, pv_s_tail, pk_m, pk_m_tail;   // pool
  CUtensorMap rk_s, rv_s, rk_m;                                     // response K, V, K
  CUtensorMap pv_m, pv_m_tail, rv_m;   // V as 128 columns x 64 channels (256-key tile variant)
  const int32_t* part_pages;
  const int32_t* part_page_offset;
  const int32_t* part_tail_slot;
  const int64_t* part_tokens;
  const float* lse;      // [R, Hq]
  const float* delta;    // [R, Hq]
  float* dq_acc;         // [R, Hq, D] fp32 running sum over parts, unscaled (dQ pass)
  __nv_bfloat16* dq;     // [R, Hq, D] final result, written by the last part of every chain
  int* ctl;              // hand-over control words (dQ pass)
  __nv_bfloat16* out;    // dk_resp or dv_resp [R, Hkv, D] (dK / dV pass over the response block)
  float* grad;           // dK / dV pass: fp32 gradient pages [slot, page, Hkv, D]; accumulated into (suffix
                         // keys) or added to `out` (response keys, when not NULL)
  int32_t* status;
  long long* timing;     // diagnostic builds only
  int R, Hq, Hkv, g, parts, pg_shift, tiles_per_head, nq_tiles, num_phys_pages;
  // dQ pass of a short response (single-CTA kernel): Q tiles of bt tokens x bh heads (RowTiling)
  int bt, bh, tiles_tok;
  // single-CTA dQ kernel, one tile per KV group: the key tiles of a KV head are cut into dq1_ranges equal
  // ranges, one CTA each; every CTA writes its fp32 sum to dq_split [dq1_ranges, R, Hq, D] and a reduce
  // kernel adds them (a chain of links per KV group would run its folds one after the other at the end
  // of a launch in which all CTAs finish together)
  float* dq_split;
  int a_slab_bytes;   // single-CTA dQ kernel: bytes of one 64-channel group of the tile's Q (dO) rows
  int dq1_ring;       // ... and the number of 32 KB ring slots that fit beside them
  int dq1_ranges;     // ... with dq_split: CTAs (= partials) per KV head
  int no_resp;   // dQ pass: the response block is left out
  // dK / dV pass: keys of a suffix block (1) read through pages [key_page_off, ..) of part_pages,
  // key_tokens of them, first gradient slot grad_slot0; or the response block (0)
  int keys_paged, key_page_off, key_tokens, grad_slot0;
  float scale, scale_log2;
};

#ifdef LS_TIMING
#define LS_BTWAIT(acc, expr) ([&] { const long long t0_ = clock64(); const bool r_ = (expr); (acc) += clock64() - t0_; return r_; }())
#define LS_BTDUMP(slot, val) do { if (p.timing && it.link == 1 && it.kvh == 0 && it.pairi == 0 && rank == 0) p.timing[(slot)] = (val); } while (0)
#else
#define LS_BTWAIT(acc, expr) (expr)
#define LS_BTDUMP(slot, val) do { } while (0)
#endif

constexpr int kBwdThreads = 320;        // producer warp, MMA warp, 8 elementwise warps (2 threads per row)
constexpr int kDq1Threads = 576;        // single-CTA dQ kernel: 16 elementwise warps (4 threads per row)
constexpr int kBwdChunk = 32768;        // 128 columns x 128 channels
constexpr float kLog2e = 1.4426950408889634f;

template <int D>
struct BwdCfg {
  static constexpr int SLABS = D / 64;            // 64-channel groups of the resident operands
  static constexpr int NC = D / 128;              // chunks per streamed operand and tile
  static constexpr int RING = (D == 128) ? 4 : 3;
  static constexpr int A_BYTES = 2 * SLABS * 16384;
  static constexpr int SMEM_BYTES = 1024 + A_BYTES + RING * kBwdChunk + 512;
};

// dK / dV of 128 keys: the 128-wide column tile halves how often the resident operand is
// re-read from shared memory per column (a 64-wide S/T MMA is bound by that re-read, not by the
// tensor pipe).  TMEM: ACC [0, D), S [D, D+128), T [D+128, D+256).
template <int D, int MODE>
__global__ void __launch_bounds__(kBwdThreads, 1) bwd_kv_kernel(const __grid_constant__ BwdParams p) {
  using C = BwdCfg<D>;
  constexpr bool HAS_T = (MODE != MODE_DV);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* a1_smem = smem;
  uint8_t* a2_smem = smem + C::SLABS * 16384;
  uint8_t* ring = smem + C::A_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + C::RING * kBwdChunk);
  uint64_t* a_full = bars;
  uint64_t* full = bars + 1;
  uint64_t* empty = full + C::RING;
  uint64_t* s_full = empty + C::RING;    // S of a tile is in TMEM
  uint64_t* t_full = s_full + 1;         // T of a tile is in TMEM (S only in mode DV)
  uint64_t* e_full = t_full + 1;         // [4] quarter q of E is in TMEM
  uint64_t* acc_final = e_full + 4;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_final + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- work item: 128 keys of one KV head; columns = (head of the group, 128-query tile)
  const int key_tiles = p.keys_paged ? (p.key_tokens + 127) / 128 : p.tiles_per_head;
  const int kvh = blockIdx.x / key_tiles;
  const int row0 = (blockIdx.x % key_tiles) * 128;      // first key of the tile
  const int tt_min = p.keys_paged ? 0 : row0 / 128;     // response keys are seen by queries t >= j only
  const int n_tt = p.tiles_per_head - tt_min;
  const int n_tiles = p.g * n_tt;
  const int n_keys = p.keys_paged ? p.key_tokens : p.R;

  if (threadIdx.x == 0) {
    mbar_init(a_full, 1);
    for (int i = 0; i < C::RING; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    mbar_init(s_full, 1);
    mbar_init(t_full, 1);
    for (int i = 0; i < 4; ++i) mbar_init(&e_full[i], 256);
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
  const uint32_t tmem_s = tmem_base + D;
  const uint32_t tmem_t = tmem_base + D + 128;

  if (warp == 0) {
    // =========================================================== producer (one thread)
    if (lane == 0 && n_tiles > 0) {
      mbar_arrive_expect_tx(a_full, (HAS_T ? 2 : 1) * C::SLABS * 16384);
      if (!p.keys_paged) {
        for (int c = 0; c < C::SLABS; ++c) {
          tma_load_5d(a1_smem + c * 16384, &p.a1_map, a_full, 0, row0, c, kvh, 0);
          if (HAS_T) tma_load_5d(a2_smem + c * 16384, &p.a2_map, a_full, 0, row0, c, kvh, 0);
        }
      } else {
        // keys of a suffix block through its pages: one 128-token box, or two 64-token pages
        const int32_t* pages = p.part_pages + p.key_page_off;
        const int n_pages = (p.key_tokens + (1 << p.pg_shift) - 1) >> p.pg_shift;
        const int pg_mask = (1 << p.pg_shift) - 1;
        const int boxes = p.pg_shift == 6 ? 2 : 1;
        for (int b = 0; b < boxes; ++b) {
          const int tok = row0 + b * 64;
          const int ps = tok >> p.pg_shift;
          const int page = ps < n_pages ? __ldg(pages + ps) : p.num_phys_pages;   // past the end: zeros
          for (int c = 0; c < C::SLABS; ++c) {
            tma_load_5d(a1_smem + c * 16384 + b * 8192, &p.a1_map, a_full, 0, tok & pg_mask, c, kvh, page);
            if (HAS_T) tma_load_5d(a2_smem + c * 16384 + b * 8192, &p.a2_map, a_full, 0, tok & pg_mask, c, kvh, page);
          }
        }
      }
      uint32_t slot = 0, phase = 0, issued = 0;
      bool ok = true;
      // one chunk: 128 columns x channels [128 c, 128 c + 128) of source `which` (0: B1, 1: B2, 2: B3)
      auto load = [&](int which, int i, int c) {
        ok = ok && mbar_wait(&empty[slot], phase ^ 1, abort_flag);
        if (ok) {
          mbar_arrive_expect_tx(&full[slot], kBwdChunk);
          uint8_t* dst = ring + slot * kBwdChunk;
          const int hh = kvh * p.g + i / n_tt;
          const int tq = (tt_min + i % n_tt) * 128;
          const CUtensorMap* m = which == 0 ? &p.b1r_map : which == 1 ? &p.b2r_map : &p.b3r_map;
          tma_load_5d(dst, m, &full[slot], 0, tq, 2 * c, hh, 0);
        }
        ++issued;
        if (++slot == (uint32_t)C::RING) { slot = 0; phase ^= 1; }
      };
      auto load_st = [&](int i) {
        for (int c = 0; c < C::NC; ++c) load(0, i, c);
        if (HAS_T)
          for (int c = 0; c < C::NC; ++c) load(1, i, c);
      };
      // chunk order = consumption order: ST(0) [M(i) ST(i+1)] ...
      load_st(0);
      for (int i = 0; i < n_tiles; ++i) {
        for (int c = 0; c < C::NC; ++c) load(2, i, c);
        if (i + 1 < n_tiles) load_st(i + 1);
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
      constexpr uint32_t idesc_st = make_idesc(128, 128, 0, 0);
      constexpr uint32_t idesc_acc = make_idesc(128, 128, 0, 1);
      constexpr uint32_t hi = sdesc_hi(1024);
      const uint32_t a1_lo = sdesc_lo(smem_u32(a1_smem), 16), a2_lo = sdesc_lo(smem_u32(a2_smem), 16);
      const uint32_t ring_k_lo = sdesc_lo(smem_u32(ring), 16);       // K-major view of a chunk
      const uint32_t ring_m_lo = sdesc_lo(smem_u32(ring), 16384);    // MN-major view: 16 KB group pitch
      uint32_t slot = 0, phase = 0;
      bool ok = mbar_wait(a_full, 0, abort_flag);
      auto advance = [&]() {
        if (++slot == (uint32_t)C::RING) { slot = 0; phase ^= 1; }
      };
      auto issue_st = [&](int i) {
#pragma unroll
        for (int op = 0; op < (HAS_T ? 2 : 1); ++op) {
          const uint32_t a_lo = op == 0 ? a1_lo : a2_lo;
          const uint32_t d = op == 0 ? tmem_s : tmem_t;
#pragma unroll
          for (int c = 0; c < C::NC; ++c) {
            ok = ok && mbar_wait(&full[slot], phase, abort_flag);
            if (!ok) return;
            tc_fence_after();
            const uint32_t b_lo = ring_k_lo + slot * (kBwdChunk >> 4);
#pragma unroll
            for (int s = 0; s < 2; ++s)
#pragma unroll
              for (int k = 0; k < 4; ++k)
                mma_ss(d, sdesc(a_lo + (((2 * c + s) * 16384 + k * 32) >> 4), hi),
                       sdesc(b_lo + ((s * 16384 + k * 32) >> 4), hi), idesc_st, (c | s | k) != 0);
            mma_commit(&empty[slot]);
            advance();
          }
          mma_commit(op == 0 ? s_full : t_full);
        }
        if (!HAS_T) mma_commit(t_full);
      };
      auto issue_acc = [&](int i) {
        // the NC chunks of B3 sit in consecutive ring slots starting at `slot`
        uint32_t cs[C::NC], cph[C::NC];
#pragma unroll
        for (int c = 0; c < C::NC; ++c) {
          cs[c] = slot;
          cph[c] = phase;
          advance();
        }
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) {
          ok = ok && mbar_wait(&e_full[qd], i & 1, abort_flag);
          if (!ok) return;
          tc_fence_after();
#pragma unroll
          for (int c = 0; c < C::NC; ++c) {
            if (qd == 0) {
              ok = ok && mbar_wait(&full[cs[c]], cph[c], abort_flag);
              if (!ok) return;
              tc_fence_after();
            }
            const uint32_t b_lo = ring_m_lo + cs[c] * (kBwdChunk >> 4);
#pragma unroll
            for (int kk = 0; kk < 2; ++kk)
              mma_ts(tmem_acc + c * 128, tmem_s + (2 * qd + kk) * 8, sdesc(b_lo + (((2 * qd + kk) * 2048) >> 4), hi),
                     idesc_acc, (i | qd | kk) != 0);
            if (qd == 3) mma_commit(&empty[cs[c]]);
          }
        }
        if (i == n_tiles - 1) mma_commit(acc_final);
      };
      if (ok) issue_st(0);
      for (int i = 0; i < n_tiles && ok; ++i) {
        issue_acc(i);
        if (ok && i + 1 < n_tiles) issue_st(i + 1);
      }
    }
  } else {
    // =========================================================== elementwise + epilogue
    // two threads per row: warps 2-5 take the lower 16 columns of every 32-column quarter,
    // warps 6-9 the upper 16 (a warp may only touch the TMEM lanes of its quadrant, warp % 4)
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;
    const int row = quad * 32 + lane;
    const int r_idx = row0 + row;                 // key j
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    const bool row_ok = r_idx < n_keys;
    bool ok = true;
    for (int i = 0; i < n_tiles; ++i) {
      // per-column constants: lane L holds columns L + 32 q of the tile
      float cl[4] = {0.f, 0.f, 0.f, 0.f}, cd[4] = {0.f, 0.f, 0.f, 0.f};
      const int hh = kvh * p.g + i / n_tt;
      const int tq0 = (tt_min + i % n_tt) * 128;
#pragma unroll
      for (int qd = 0; qd < 4; ++qd) {
        const int tc = min(tq0 + 32 * qd + lane, p.R - 1);
        cl[qd] = __ldg(p.lse + (size_t)tc * p.Hq + hh) * kLog2e;
        if (MODE == MODE_DK) cd[qd] = __ldg(p.delta + (size_t)tc * p.Hq + hh);
      }
      // column t is visible to key row j when j <= t < R (response keys) or t < R (suffix keys)
      const bool edge = (!p.keys_paged && tq0 < row0 + 127) || (tq0 + 127 >= p.R);
      const int t_min = p.keys_paged ? 0 : r_idx;
      // ---- p = exp(s - LSE) for this thread's 4 x 16 columns, as soon as S is complete
      // (the T MMAs are still running)
      ok = ok && mbar_wait(s_full, i & 1, abort_flag);
      tc_fence_after();
      float pr[64];
#pragma unroll
      for (int qd = 0; qd < 4; ++qd) {
        uint32_t sr[16];
        tmem_ld16(tmem_s + lane_sel + 32 * qd + 16 * half, sr);
        tc_wait_ld16(sr);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float l0 = __shfl_sync(0xffffffffu, cl[qd], 16 * half + j);
          float e = ex2(fmaf(__uint_as_float(sr[j]), p.scale_log2, -l0));
          if (edge) {
            const int ta = tq0 + 32 * qd + 16 * half + j;
            if (ta < t_min || ta >= p.R) e = 0.f;
          }
          pr[16 * qd + j] = e;
        }
      }
      // E overwrites S columns that the row's other thread reads: all 256 threads must be done
      // reading S before anyone writes (named barrier 1; the T MMAs normally still run here).
      // The barrier also carries the vote on whether any wait gave up: the threads leave the
      // loop together or not at all.
      ok = bar_and(1, 256, ok);
      if (!ok) break;
      // ---- E = p (T - Delta), quarter by quarter, once T is complete
      ok = mbar_wait(t_full, i & 1, abort_flag);     // a failure here is voted on in the next round
      tc_fence_after();
#pragma unroll
      for (int qd = 0; qd < 4; ++qd) {
        uint32_t pk[8];
        if (HAS_T) {
          uint32_t tr[16];
          tmem_ld16(tmem_t + lane_sel + 32 * qd + 16 * half, tr);
          tc_wait_ld16(tr);
#pragma unroll
          for (int j = 0; j < 16; j += 2) {
            const float d0 = __shfl_sync(0xffffffffu, cd[qd], 16 * half + j);
            const float d1 = __shfl_sync(0xffffffffu, cd[qd], 16 * half + j + 1);
            pk[j >> 1] = pack_bf16(pr[16 * qd + j] * (__uint_as_float(tr[j]) - d0),
                                   pr[16 * qd + j + 1] * (__uint_as_float(tr[j + 1]) - d1));
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; j += 2) pk[j >> 1] = pack_bf16(pr[16 * qd + j], pr[16 * qd + j + 1]);
        }
        // quarter q of E (bf16 pairs) lands in columns [16 q, 16 q + 16) of the S region, whose
        // fp32 contents every thread has already pulled into registers
        tmem_st8(tmem_s + lane_sel + 16 * qd + 8 * half, pk);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(&e_full[qd]);
      }
    }
    if (n_tiles > 0 && ok) ok = mbar_wait(acc_final, 0, abort_flag);
    if (n_tiles > 0 && ok) {
      tc_fence_after();
      const float out_scale = (MODE == MODE_DK) ? p.scale : 1.0f;
      // gradient page row of this key: pages are indexed by suffix slot
      float* grow = nullptr;
      if (p.grad) {
        const int pg = 1 << p.pg_shift;
        const int kk = min(r_idx, n_keys - 1);
        grow = p.grad + ((((size_t)p.grad_slot0 + (kk >> p.pg_shift)) * pg + (kk & (pg - 1))) * p.Hkv + kvh) * D;
      }
#pragma unroll 1
      for (int c = half * (D / 2); c < (half + 1) * (D / 2); c += 32) {
        uint32_t o[32];
        tmem_ld32(tmem_acc + lane_sel + c, o);
        tc_wait_ld32(o);
        if (row_ok) {
          float v[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(o[j]) * out_scale;
          if (grow) {
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              const float4 gv = *reinterpret_cast<const float4*>(grow + c + j);
              v[j] += gv.x; v[j + 1] += gv.y; v[j + 2] += gv.z; v[j + 3] += gv.w;
            }
          }
          if (p.keys_paged) {
            // suffix keys: the sum stays in the fp32 gradient page (this CTA alone owns these rows)
#pragma unroll
            for (int j = 0; j < 32; j += 4)
              *reinterpret_cast<float4*>(grow + c + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
          } else {
            __nv_bfloat16* dst = p.out + ((size_t)r_idx * p.Hkv + kvh) * D + c;
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              uint4 w;
              w.x = pack_bf16(v[j], v[j + 1]);
              w.y = pack_bf16(v[j + 2], v[j + 3]);
              w.z = pack_bf16(v[j + 4], v[j + 5]);
              w.w = pack_bf16(v[j + 6], v[j + 7]);
              *reinterpret_cast<uint4*>(dst + j) = w;
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

// Row-thread wait of the dQ kernels: returns the warp's common answer.
__device__ __forceinline__ bool bwd_wait_warp(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
}

// Work item of the dQ pass: link 0 is the causal response block, links 1.. are the prefix
// sub-shards and then the suffix blocks; the links of one row tile are summed in that order.
struct DqItem {
  int kvh, link, part, pairi;
  bool is_resp;
};
__device__ __forceinline__ DqItem dq_item(const BwdParams& p, int idx, int npairs) {
  DqItem it;
  it.pairi = idx % npairs;
  idx /= npairs;
  it.link = idx % (p.parts + 1);
  it.kvh = idx / (p.parts + 1);
  it.is_resp = it.link == 0;
  it.part = it.is_resp ? p.parts : it.link - 1;
  return it;
}

// One row thread's share of the dQ epilogue: NCOL accumulator columns of its row are added
// to the running fp32 sum (fold), stored as the first term, or -- last link -- scaled and
// written as bf16.  An empty part in the middle of a chain leaves the sum untouched.
template <int NCOL>
__device__ __forceinline__ void dq_store_row(uint32_t tmem_row, bool have_acc, bool fold, bool last, float scale,
                                             float* acc_dst, __nv_bfloat16* dq_dst, bool row_ok) {
  if (!have_acc && fold && !last) return;
  const uint64_t pol = last ? l2_policy_evict_first() : l2_policy_evict_last();
#pragma unroll 1
  for (int c = 0; c < NCOL; c += 32) {
    uint32_t o[32];
    if (have_acc) {
      tmem_ld32(tmem_row + c, o);
      tc_wait_ld32(o);
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) o[j] = 0u;
    }
    if (row_ok) {
      float4 run[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        run[j] = fold ? ld_cg_hint(reinterpret_cast<const float4*>(acc_dst + c) + j, pol) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float4 v;
        v.x = run[j].x + __uint_as_float(o[4 * j]);
        v.y = run[j].y + __uint_as_float(o[4 * j + 1]);
        v.z = run[j].z + __uint_as_float(o[4 * j + 2]);
        v.w = run[j].w + __uint_as_float(o[4 * j + 3]);
        if (last) {
          uint2 pk;
          pk.x = pack_bf16(v.x * scale, v.y * scale);
          pk.y = pack_bf16(v.z * scale, v.w * scale);
          *(reinterpret_cast<uint2*>(dq_dst + c) + j) = pk;
        } else {
          st_hint(reinterpret_cast<float4*>(acc_dst + c) + j, v, pol);
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------
// dQ pass on CTA pairs (cta_group::2), 128-key tiles.  Two neighbouring SMs take two Q tiles of
// the same (KV head, part) and stream the keys once between them: each CTA loads only half of
// every K/V chunk (64 of the 128 keys for S and T, half of the channels for ACC).  One thread of
// the even CTA issues all MMAs (256 rows); completions are multicast to both CTAs' barriers;
// the odd CTA's row threads report to the even CTA's barriers.
// TMEM: ACC [0, D), S [D, D+128), T [D+128, D+256).  E (bf16) is written over T, not over S, so
// the S buffer is free as soon as the row threads have pulled it and the tensor pipe runs
//     S(0) T(0) | S(i+1)  ACC(i)  T(i+1) | ...
// with S(i+1) overlapping the row threads' E(i) and ACC(i) / T(i+1) overlapping their p(i+1).
// ---------------------------------------------------------------------------------
constexpr int kDq2Chunk = 16384;

template <int D>
struct Dq2Cfg {
  static constexpr int SLABS = D / 64;
  static constexpr int NC = D / 128;
  static constexpr int RING = (D == 128) ? 8 : 6;
  static constexpr int A_BYTES = 2 * SLABS * 16384;
  static constexpr int SMEM_BYTES = 1024 + A_BYTES + RING * kDq2Chunk + 512;
};

template <int D>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kBwdThreads, 1)
    bwd_dq2_kernel(const __grid_constant__ BwdParams p) {
  using C = Dq2Cfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* a1_smem = smem;
  uint8_t* a2_smem = smem + C::SLABS * 16384;
  uint8_t* ring = smem + C::A_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + C::RING * kDq2Chunk);
  uint64_t* a_full = bars;               // (even CTA) both CTAs' resident operands landed
  uint64_t* full = bars + 1;             // (even CTA) both halves of a chunk landed
  uint64_t* empty = full + C::RING;      // (each CTA) chunk consumed
  uint64_t* s_full = empty + C::RING;    // (each CTA) S in TMEM
  uint64_t* s_read = s_full + 1;         // (even CTA) every row thread of both CTAs has pulled S: 16 warp arrivals
  uint64_t* t_full = s_read + 1;         // (each CTA) T in TMEM
  uint64_t* e_full = t_full + 1;         // [4] (even CTA) quarter of E in both CTAs' TMEM: 16 warp arrivals
  uint64_t* acc_final = e_full + 4;      // (each CTA)
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_final + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  int* work_idx = const_cast<int*>(abort_flag) + 1;   // (even CTA) the pair's work item

  long long tw0 = 0, tw1 = 0, tw2 = 0;   // wait-time accumulators (only used with LS_TIMING)
  (void)tw0; (void)tw1; (void)tw2;
  const long long t_kernel0 = clock64();
  (void)t_kernel0;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    mbar_init(a_full, 1);
    for (int i = 0; i < C::RING; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    mbar_init(s_full, 1);
    mbar_init(s_read, 16);
    mbar_init(t_full, 1);
    for (int i = 0; i < 4; ++i) mbar_init(&e_full[i], 16);
    mbar_init(acc_final, 1);
    *abort_flag = 0;
    // work items are handed out in launch order of the pairs that ask (see chain_wait)
    if (leader) *work_idx = atomicAdd(p.ctl, 1);
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_holder, 512);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                      // both CTAs' barriers exist before any remote signal
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  const uint32_t tmem_acc = tmem_base;
  const uint32_t tmem_s = tmem_base + D;
  const uint32_t tmem_t = tmem_base + D + 128;

  // ---- work item of the pair, and this CTA's Q tile
  const int npairs = (p.nq_tiles + 1) / 2;
  const DqItem it = dq_item(p, (int)ld_shared_cluster_u32(mapa_u32(smem_u32(work_idx), 0)), npairs);
  const int pairi = it.pairi, part = it.part, kvh = it.kvh;
  const bool is_resp = it.is_resp;
  auto tile_of = [&](int qt, int& hh, int& r0) {
    if (qt < p.nq_tiles) {
      hh = kvh * p.g + qt / p.tiles_per_head;
      r0 = (qt % p.tiles_per_head) * 128;
    } else {                                 // odd tile count: the pair's second CTA works on zero rows
      hh = kvh * p.g + p.g - 1;
      r0 = p.tiles_per_head * 128;           // token coordinate past R: TMA delivers zeros
    }
  };
  const int qtile = 2 * pairi + (int)rank;
  int h, row0, h_o, row0_o;
  tile_of(qtile, h, row0);
  tile_of(2 * pairi + 1 - (int)rank, h_o, row0_o);
  int64_t tokens;
  int page_off = 0, n_pages = 0, tail_slot = -1;
  if (is_resp) {
    tokens = p.no_resp ? 0 : min(p.R, max(row0, row0_o) + 128);      // both CTAs walk the longer causal range
  } else {
    tokens = p.part_tokens[part];
    page_off = p.part_page_offset[part];
    n_pages = p.part_page_offset[part + 1] - page_off;
    tail_slot = p.part_tail_slot[part];
  }
  const int n_tiles = (int)((tokens + 127) / 128);

  if (warp == 0) {
    // =========================================================== producer (one thread per CTA)
    if (lane == 0 && n_tiles > 0) {
      const int a_rows = 128;
      if (leader) mbar_arrive_expect_tx(a_full, 2 * 2 * C::SLABS * a_rows * 128);
      for (int c = 0; c < C::SLABS; ++c) {
        tma_load_5d_pair(a1_smem + c * 16384, &p.a1_map, a_full, 0, row0, c, h, 0);
        tma_load_5d_pair(a2_smem + c * 16384, &p.a2_map, a_full, 0, row0, c, h, 0);
      }
      const int32_t* pages = p.part_pages + page_off;
      const int pg_mask = (1 << p.pg_shift) - 1;
      const bool small_pages = !is_resp && p.pg_shift == 6;
      auto fetch = [&](int ps) -> int {
        if (is_resp) return 0;
        return (ps < n_pages) ? __ldg(pages + ps) : p.num_phys_pages;   // past the end: TMA fills zeros
      };
      uint32_t slot = 0, phase = 0, issued = 0;
      bool ok = true;
      // `which` 0: this CTA's 64 keys of K for S; 1: of V for T; 2: this CTA's 64 channels of K for ACC
      auto load = [&](int which, int i, int c, int pa, int pb) {
        ok = ok && LS_BTWAIT(tw0, mbar_wait(&empty[slot], phase ^ 1, abort_flag));
        if (ok) {
          if (leader) mbar_arrive_expect_tx(&full[slot], 2 * kDq2Chunk);
          uint8_t* dst = ring + slot * kDq2Chunk;
          const int tok = i * 128;
          if (which < 2) {
            const int tk = tok + (int)rank * 64;
            if (is_resp) {
              tma_load_5d_pair(dst, which ? &p.rv_s : &p.rk_s, &full[slot], 0, tk, 2 * c, kvh, 0);
            } else {
              const bool tail = (tk >> p.pg_shift) == tail_slot;
              const CUtensorMap* m = which ? (tail ? &p.pv_s_tail : &p.pv_s) : (tail ? &p.pk_s_tail : &p.pk_s);
              tma_load_5d_pair(dst, m, &full[slot], 0, tk & pg_mask, 2 * c, kvh, (small_pages && rank) ? pb : pa);
            }
          } else {
            // D = 256: one 256-wide MMA covers both chunks, so this CTA owns channels [128 rank, +128)
            // and chunk c is its c-th 64-channel group; D = 128: the single chunk's half `rank`
            const int grp = (C::NC == 2) ? 2 * (int)rank + c : (int)rank;
            if (is_resp) {
              tma_load_5d_pair(dst, &p.rk_m, &full[slot], 0, tok, grp, kvh, 0);
            } else if (!small_pages) {
              const bool tail = (tok >> p.pg_shift) == tail_slot;
              tma_load_5d_pair(dst, tail ? &p.pk_m_tail : &p.pk_m, &full[slot], 0, tok & pg_mask, grp, kvh, pa);
            } else {
              const int sa = tok >> 6;
              tma_load_5d_pair(dst, sa == tail_slot ? &p.pk_m_tail : &p.pk_m, &full[slot], 0, 0, grp, kvh, pa);
              tma_load_5d_pair(dst + 8192, sa + 1 == tail_slot ? &p.pk_m_tail : &p.pk_m, &full[slot], 0, 0, grp, kvh, pb);
            }
          }
        }
        ++issued;
        if (++slot == (uint32_t)C::RING) { slot = 0; phase ^= 1; }
      };
      // chunk order = consumption order: S(0) T(0) [S(i+1) ACC(i) T(i+1)] ...
      auto load_op = [&](int which, int i, int pa, int pb) {
        for (int c = 0; c < C::NC; ++c) load(which, i, c, pa, pb);
      };
      const int sh = p.pg_shift - 7;
      auto slot_of = [&](int i) { return small_pages ? 2 * i : (i >> sh); };
      int pa0 = fetch(slot_of(0)), pb0 = small_pages ? fetch(1) : pa0;
      int pa1 = fetch(slot_of(1)), pb1 = small_pages ? fetch(3) : pa1;
      load_op(0, 0, pa0, pb0);
      load_op(1, 0, pa0, pb0);
      for (int i = 0; i < n_tiles; ++i) {
        const int pa2 = fetch(slot_of(i + 2)), pb2 = small_pages ? fetch(2 * i + 5) : pa2;
        if (i + 1 < n_tiles) load_op(0, i + 1, pa1, pb1);
        load_op(2, i, pa0, pb0);
        if (i + 1 < n_tiles) load_op(1, i + 1, pa1, pb1);
        pa0 = pa1; pb0 = pb1; pa1 = pa2; pb1 = pb2;
      }
      LS_BTDUMP(0, tw0);
      LS_BTDUMP(1, clock64() - t_kernel0);
      if (*abort_flag && leader) {   // aborted: wait (bounded) for the copies credited to this CTA's barriers
        for (uint32_t s = 0; s < (uint32_t)C::RING && s < issued; ++s) {
          const uint32_t last = ((issued - 1 - s) / C::RING) * C::RING + s;
          const uint64_t t_start = globaltimer_ns();
          while (!mbar_try_wait(&full[s], (last / C::RING) & 1, 1000) && globaltimer_ns() - t_start < 100000000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // =========================================================== MMA issuer (one thread of the even CTA)
    if (leader && lane == 0 && n_tiles > 0) {
      constexpr uint32_t idesc_st = make_idesc(256, 128, 0, 0);
      constexpr uint32_t idesc_acc = make_idesc(256, 128, 0, 1);
      constexpr uint32_t hi = sdesc_hi(1024);
      const uint32_t a1_lo = sdesc_lo(smem_u32(a1_smem), 16), a2_lo = sdesc_lo(smem_u32(a2_smem), 16);
      const uint32_t ring_lo = sdesc_lo(smem_u32(ring), 16);
      constexpr uint32_t idesc_acc2 = make_idesc(256, 256, 0, 1);
      const uint32_t ring2_lo = sdesc_lo(smem_u32(ring), kDq2Chunk);   // MN-major, two 64-channel groups one slot apart
      uint32_t slot = 0, phase = 0;
      bool ok = mbar_wait(a_full, 0, abort_flag);
      auto advance = [&]() {
        if (++slot == (uint32_t)C::RING) { slot = 0; phase ^= 1; }
      };
      // S = Q K^T (op 0) or T = dO V^T (op 1) of tile i
      auto issue_op = [&](int op) {
        {
          const uint32_t a_lo = op == 0 ? a1_lo : a2_lo;
          const uint32_t d = op == 0 ? tmem_s : tmem_t;
#pragma unroll
          for (int c = 0; c < C::NC; ++c) {
            ok = ok && LS_BTWAIT(tw0, mbar_wait(&full[slot], phase, abort_flag));
            if (!ok) return;
            tc_fence_after();
            const uint32_t b_lo = ring_lo + slot * (kDq2Chunk >> 4);
#pragma unroll
            for (int s = 0; s < 2; ++s)
#pragma unroll
              for (int k = 0; k < 4; ++k)
                mma_ss_pair(d, sdesc(a_lo + (((2 * c + s) * 16384 + k * 32) >> 4), hi),
                            sdesc(b_lo + ((s * 8192 + k * 32) >> 4), hi), idesc_st, (c | s | k) != 0);
            mma_commit_pair(&empty[slot]);
            advance();
          }
          mma_commit_pair(op == 0 ? s_full : t_full);
        }
      };
      auto issue_acc = [&](int i) {
        uint32_t cs[C::NC], cph[C::NC];
#pragma unroll
        for (int c = 0; c < C::NC; ++c) {
          cs[c] = slot;
          cph[c] = phase;
          advance();
        }
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) {
          ok = ok && LS_BTWAIT(tw1, mbar_wait(&e_full[qd], i & 1, abort_flag));
          if (!ok) return;
          tc_fence_after();
          if (qd == 0) {
#pragma unroll
            for (int c = 0; c < C::NC; ++c) {
              ok = ok && LS_BTWAIT(tw2, mbar_wait(&full[cs[c]], cph[c], abort_flag));
              if (!ok) return;
            }
            tc_fence_after();
          }
          if (C::NC == 2) {
            // D = 256: the two 64-channel groups sit in adjacent slots (every operand takes two slots
            // of a ring of six, so a pair never wraps): one 256-wide MMA per 16 keys
            const uint32_t b_lo = ring2_lo + cs[0] * (kDq2Chunk >> 4);
#pragma unroll
            for (int kk = 0; kk < 2; ++kk)
              mma_ts_pair(tmem_acc, tmem_t + (2 * qd + kk) * 8, sdesc(b_lo + (((2 * qd + kk) * 2048) >> 4), hi),
                          idesc_acc2, (i | qd | kk) != 0);
          } else {
#pragma unroll
            for (int c = 0; c < C::NC; ++c) {
              const uint32_t b_lo = ring_lo + cs[c] * (kDq2Chunk >> 4);
#pragma unroll
              for (int kk = 0; kk < 2; ++kk)
                mma_ts_pair(tmem_acc + c * 128, tmem_t + (2 * qd + kk) * 8,
                            sdesc(b_lo + (((2 * qd + kk) * 2048) >> 4), hi), idesc_acc, (i | qd | kk) != 0);
            }
          }
          if (qd == 3) {
#pragma unroll
            for (int c = 0; c < C::NC; ++c) mma_commit_pair(&empty[cs[c]]);
          }
        }
        if (i == n_tiles - 1) mma_commit_pair(acc_final);
      };
      // E overwrites T (not S), so S of the next tile only waits for the row threads to have pulled S:
      // the tensor pipe runs S(i+1) while the row threads form E(i), then ACC(i), then T(i+1).
      if (ok) issue_op(0);
      if (ok) issue_op(1);
      for (int i = 0; i < n_tiles && ok; ++i) {
        if (i + 1 < n_tiles) {
          ok = ok && LS_BTWAIT(tw0, mbar_wait(s_read, i & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
          issue_op(0);
        }
        if (ok) issue_acc(i);
        if (ok && i + 1 < n_tiles) issue_op(1);
      }
      LS_BTDUMP(8, tw0);
      LS_BTDUMP(9, tw1);
      LS_BTDUMP(10, tw2);
      LS_BTDUMP(11, clock64() - t_kernel0);
    }
  } else {
    // =========================================================== elementwise + epilogue (both CTAs)
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;
    const int row = quad * 32 + lane;
    // this thread's (token, head): 128 tokens of one head
    const int r_idx = row0 + row;
    const int hr = h;
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    const bool tile_ok = qtile < p.nq_tiles;
    const bool row_ok = tile_ok && r_idx < p.R;
    const size_t ri = (size_t)min(r_idx, p.R - 1) * p.Hq + hr;
    bool ok = true;
    if (n_tiles > 0) {
      const float lse2_row = p.lse[ri] * kLog2e;
      const float delta_row = p.delta[ri];
      const int64_t lim = is_resp ? (int64_t)min(r_idx, p.R - 1) : tokens - 1;
      const uint32_t s_read_remote = mapa_u32(smem_u32(s_read), 0);
      uint32_t e_remote[4];
#pragma unroll
      for (int qd = 0; qd < 4; ++qd) e_remote[qd] = mapa_u32(smem_u32(&e_full[qd]), 0);
      for (int i = 0; i < n_tiles; ++i) {
        const int key0 = i * 128;
        const bool edge = __any_sync(0xffffffffu, (int64_t)key0 + 127 > lim);
        // No thread leaves this loop on its own: a wait that gave up is remembered in `ok` and put
        // to the vote at the tile's named barrier, where all 256 leave together.
        ok = ok && LS_BTWAIT(tw0, mbar_wait(s_full, i & 1, abort_flag));
        tc_fence_after();
        // p = exp(s - LSE) for this thread's 4 x 16 columns; once S is in registers the next tile's
        // S may overwrite the buffer
        uint32_t sr[64];
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) tmem_ld16(tmem_s + lane_sel + 32 * qd + 16 * half, sr + 16 * qd);
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) tc_wait_ld16(sr + 16 * qd);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(s_read_remote);
        float pr[64];
#pragma unroll
        for (int j = 0; j < 64; ++j) {
          float e = ex2(fmaf(__uint_as_float(sr[j]), p.scale_log2, -lse2_row));
          if (edge && (int64_t)key0 + 32 * (j >> 4) + 16 * half + (j & 15) > lim) e = 0.f;
          pr[j] = e;
        }
        // T of the tile, all of it into registers: E (bf16) goes over T's columns, which the row's
        // other thread reads too, so every T read of the CTA comes before any E write (named barrier 1)
        ok = ok && LS_BTWAIT(tw1, mbar_wait(t_full, i & 1, abort_flag));
        tc_fence_after();
        uint32_t tr[64];
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) tmem_ld16(tmem_t + lane_sel + 32 * qd + 16 * half, tr + 16 * qd);
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) tc_wait_ld16(tr + 16 * qd);
        ok = bar_and(1, 256, ok);
        if (!ok) break;
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) {
          uint32_t pk[8];
#pragma unroll
          for (int j = 0; j < 16; j += 2)
            pk[j >> 1] = pack_bf16(pr[16 * qd + j] * (__uint_as_float(tr[16 * qd + j]) - delta_row),
                                   pr[16 * qd + j + 1] * (__uint_as_float(tr[16 * qd + j + 1]) - delta_row));
          // quarter q of E (bf16 pairs) lands in columns [16 q, 16 q + 16) of the T region
          tmem_st8(tmem_t + lane_sel + 16 * qd + 8 * half, pk);
          tc_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(e_remote[qd]);   // one arrival per warp, at the even CTA
        }
      }
      if (threadIdx.x == 64) {
        LS_BTDUMP(16, tw0);
        LS_BTDUMP(17, tw1);
        LS_BTDUMP(18, clock64() - t_kernel0);
      }
      ok = __all_sync(0xffffffffu, ok);
      if (ok) ok = bwd_wait_warp(acc_final, 0, abort_flag);
      if (ok) tc_fence_after();
    }
    // ---- epilogue: add this part's sum to the running dQ of the row tile, in link order
    const bool fold = it.link > 0, last = it.link == p.parts;
    int* counter = p.ctl + kChainHeaderInts + kvh * p.nq_tiles + min(qtile, p.nq_tiles - 1);
    if (tile_ok) {
      if (ok && fold) ok = __all_sync(0xffffffffu, chain_wait(counter, it.link, p.ctl, abort_flag));
      if (ok)
        dq_store_row<D / 2>(tmem_acc + lane_sel + half * (D / 2), n_tiles > 0, fold, last, p.scale,
                            p.dq_acc + ri * D + half * (D / 2), p.dq + ri * D + half * (D / 2), row_ok);
      const bool all_ok = bar_and(2, 256, ok);     // every row of the tile is written
      if (row == 0 && half == 0 && all_ok) chain_publish(counter, it.link + 1);
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // neither CTA leaves while the other may still touch its shared memory
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 512);
  }
  if (threadIdx.x == 0 && *abort_flag) {
    if (p.status) atomicExch(p.status, (int)LS_ERR_TIMEOUT);
    st_relaxed_gpu(p.ctl + 1, 1);    // ends every other chain wait of this launch
  }
}


// ---------------------------------------------------------------------------------
// dQ pass for short responses: the rows of a Q tile (bt tokens x bh heads of one KV group) stay in
// shared memory and the keys stream past once, so the pass is bound by HBM, not by the tensor pipe.
// A single CTA per work item (a pair would spend half of every 256-row MMA on rows that do not
// exist), 128-key tiles, E written over T so that the tensor pipe runs S(i+1) while the row threads
// form E(i):   S(0) T(0) | S(i+1)  ACC(i)  T(i+1) | ...
// TMEM: ACC [0, D), S [D, D+128), T [D+128, D+256).  Chunks of 32 KB: 128 keys x 128 channels.
//
// Work.  A KV group of several tiles: one item per (KV head, link, tile), the links of a tile summed
// through the running dQ in link order.  A KV group of ONE tile (p.dq_split): the key tiles of all
// links of a KV head, laid end to end, are cut into p.dq1_ranges equal ranges, one CTA each (a range
// may cross link boundaries); every CTA writes one fp32 partial and a reduce kernel adds them.  With
// one item per (KV head, part) the 4 x 65 items of the 2M prefix ran as two waves on 148 SMs.
// ---------------------------------------------------------------------------------
struct Dq1Cursor {      // a position in the CTA's list of key tiles
  int link, i, n;       // link (0 = response block, 1.. = parts), tile of the link, tiles of the link
  int left;             // tiles of the list from here on, this one included
  bool is_resp;
  int64_t tokens;
  int page_off, n_pages, tail_slot;
};
__device__ __forceinline__ void dq1_link(const BwdParams& p, int resp_tokens, Dq1Cursor& c) {
  c.is_resp = c.link == 0;
  if (c.is_resp) {
    c.tokens = resp_tokens;
    c.page_off = c.n_pages = 0;
    c.tail_slot = -1;
  } else {
    const int part = c.link - 1;
    c.tokens = p.part_tokens[part];
    c.page_off = p.part_page_offset[part];
    c.n_pages = p.part_page_offset[part + 1] - c.page_off;
    c.tail_slot = p.part_tail_slot[part];
  }
  c.n = (int)((c.tokens + 127) / 128);
}
__device__ __forceinline__ void dq1_next(const BwdParams& p, int resp_tokens, Dq1Cursor& c) {
  if (--c.left <= 0) return;
  ++c.i;
  while (c.i >= c.n && c.link < p.parts) {     // left > 0: a later link holds the tile
    ++c.link;
    dq1_link(p, resp_tokens, c);
    c.i = 0;
  }
}

template <int D>
__global__ void __launch_bounds__(kDq1Threads, 1) bwd_dq1_kernel(const __grid_constant__ BwdParams p) {
  using C = BwdCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  // Q and dO keep only the rows of the tile (padded to 8): the 128-row MMAs read on into whatever
  // follows, which yields rows nobody stores; the ring gets the shared memory this frees
  const uint32_t slab = (uint32_t)p.a_slab_bytes;     // one 64-channel group of the resident rows
  const uint32_t nring = (uint32_t)p.dq1_ring;
  uint8_t* a1_smem = smem;
  uint8_t* a2_smem = smem + C::SLABS * slab;
  uint8_t* ring = smem + 2 * C::SLABS * slab;
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + nring * kBwdChunk);
  uint64_t* a_full = bars;
  uint64_t* full = bars + 1;
  uint64_t* empty = full + nring;
  uint64_t* s_full = empty + nring;      // S of a tile is in TMEM
  uint64_t* s_read = s_full + 1;         // every row thread has pulled S
  uint64_t* t_full = s_read + 1;         // T of a tile is in TMEM
  uint64_t* e_full = t_full + 1;         // [4] quarter q of E is in TMEM
  uint64_t* acc_final = e_full + 4;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_final + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  int* work = const_cast<int*>(abort_flag) + 1;      // [4] ticket, first link, first tile, tiles of the list

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(a_full, 1);
    for (uint32_t i = 0; i < nring; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    mbar_init(s_full, 1);
    mbar_init(s_read, 512);
    mbar_init(t_full, 1);
    for (int i = 0; i < 4; ++i) mbar_init(&e_full[i], 128);
    mbar_init(acc_final, 1);
    *abort_flag = 0;
    const int widx = atomicAdd(p.ctl, 1);      // work items in launch order of the CTAs that ask (see chain_wait)
    work[0] = widx;
    if (p.dq_split) {
      // range widx % dq1_ranges of the KV head's key tiles, all links end to end
      const int resp_tokens = p.no_resp ? 0 : min(p.R, p.bt);
      auto tiles_of = [&](int link) -> int64_t {
        return ((link == 0 ? (int64_t)resp_tokens : p.part_tokens[link - 1]) + 127) / 128;
      };
      int64_t total = 0;
      for (int link = 0; link <= p.parts; ++link) total += tiles_of(link);
      const int c = widx % p.dq1_ranges;
      const int64_t v0 = total * c / p.dq1_ranges, v1 = total * (c + 1) / p.dq1_ranges;
      int link = 0;
      int64_t v = 0;
      for (; link < p.parts; ++link) {
        const int64_t n = tiles_of(link);
        if (v0 < v + n) break;
        v += n;
      }
      work[1] = link;
      work[2] = (int)(v0 - v);
      work[3] = (int)(v1 - v0);
    }
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
  const uint32_t tmem_s = tmem_base + D;
  const uint32_t tmem_t = tmem_base + D + 128;

  // ---- the CTA's rows (KV head, Q tile of bt tokens x bh heads of the KV group) and its list of key tiles
  DqItem it{};
  int range = 0;
  if (p.dq_split) {
    range = work[0] % p.dq1_ranges;
    it.kvh = work[0] / p.dq1_ranges;
    it.pairi = 0;
    it.link = work[1];
  } else {
    it = dq_item(p, work[0], p.nq_tiles);
  }
  const int kvh = it.kvh, qtile = it.pairi;
  const int h = kvh * p.g + (qtile / p.tiles_tok) * p.bh;
  const int t0 = (qtile % p.tiles_tok) * p.bt;
  const int resp_tokens = p.no_resp ? 0 : min(p.R, t0 + p.bt);
  Dq1Cursor first;
  first.link = it.link;
  dq1_link(p, resp_tokens, first);
  first.i = p.dq_split ? work[2] : 0;
  first.left = p.dq_split ? work[3] : first.n;
  const int n_tiles = first.left;
  [[maybe_unused]] const bool dump = p.dq_split ? work[0] == 0 : (it.link == 1 && kvh == 0 && qtile == 0);
  [[maybe_unused]] long long tw0 = 0, tw1 = 0, tw2 = 0, tw3 = 0;
  [[maybe_unused]] const long long t_kernel0 = clock64();
#ifdef LS_TIMING
#define LS_D1DUMP(slot, val) do { if (p.timing && dump) p.timing[(slot)] = (val); } while (0)
#else
#define LS_D1DUMP(slot, val) do { } while (0)
#endif

  if (warp == 0) {
    // =========================================================== producer (one thread)
    if (lane == 0 && n_tiles > 0) {
      mbar_arrive_expect_tx(a_full, 2 * C::SLABS * p.bt * p.bh * 128);
      for (int c = 0; c < C::SLABS; ++c) {
        tma_load_5d(a1_smem + c * slab, &p.a1_map, a_full, 0, t0, c, h, 0);
        tma_load_5d(a2_smem + c * slab, &p.a2_map, a_full, 0, t0, c, h, 0);
      }
      const int pg_mask = (1 << p.pg_shift) - 1;
      const bool pages64 = p.pg_shift == 6;      // a 128-key tile of a paged link spans two 64-token pages
      const int sh = pages64 ? 0 : (p.pg_shift - 7);
      // physical pages under a tile (past the end of the link: TMA fills zeros)
      auto pages_of = [&](const Dq1Cursor& cu, int& pa, int& pb) {
        pa = pb = 0;
        if (cu.left <= 0 || cu.is_resp) return;
        const int32_t* pages = p.part_pages + cu.page_off;
        if (pages64) {
          pa = (2 * cu.i < cu.n_pages) ? __ldg(pages + 2 * cu.i) : p.num_phys_pages;
          pb = (2 * cu.i + 1 < cu.n_pages) ? __ldg(pages + 2 * cu.i + 1) : p.num_phys_pages;
        } else {
          pa = pb = ((cu.i >> sh) < cu.n_pages) ? __ldg(pages + (cu.i >> sh)) : p.num_phys_pages;
        }
      };
      uint32_t slot = 0, phase = 0, issued = 0;
      bool ok = true;
      // one chunk: 128 keys x channels [128 c, 128 c + 128) of K (which = 0) or V (1)
      auto load = [&](int which, const Dq1Cursor& cu, int c, int pa, int pb) {
        ok = ok && LS_BTWAIT(tw0, mbar_wait(&empty[slot], phase ^ 1, abort_flag));
        if (ok) {
          mbar_arrive_expect_tx(&full[slot], kBwdChunk);
          uint8_t* dst = ring + slot * kBwdChunk;
          const int tok = cu.i * 128;
          if (cu.is_resp) {
            tma_load_5d(dst, which ? &p.b2r_map : &p.b1r_map, &full[slot], 0, tok, 2 * c, kvh, 0);
          } else if (!pages64) {
            const bool tail = (tok >> p.pg_shift) == cu.tail_slot;
            const CUtensorMap* m = which ? (tail ? &p.bv_tail : &p.bv_map) : (tail ? &p.bk_tail : &p.bk_map);
            tma_load_5d(dst, m, &full[slot], 0, tok & pg_mask, 2 * c, kvh, pa);
          } else {
            const int sa = tok >> 6;
            const CUtensorMap* ma = which ? (sa == cu.tail_slot ? &p.bv_tail : &p.bv_map)
                                          : (sa == cu.tail_slot ? &p.bk_tail : &p.bk_map);
            const CUtensorMap* mb = which ? (sa + 1 == cu.tail_slot ? &p.bv_tail : &p.bv_map)
                                          : (sa + 1 == cu.tail_slot ? &p.bk_tail : &p.bk_map);
            for (int s2 = 0; s2 < 2; ++s2) {
              tma_load_5d(dst + s2 * 16384, ma, &full[slot], 0, 0, 2 * c + s2, kvh, pa);
              tma_load_5d(dst + s2 * 16384 + 8192, mb, &full[slot], 0, 0, 2 * c + s2, kvh, pb);
            }
          }
        }
        ++issued;
        if (++slot == nring) { slot = 0; phase ^= 1; }
      };
      auto load_op = [&](int which, const Dq1Cursor& cu, int pa, int pb) {
        for (int c = 0; c < C::NC; ++c) load(which, cu, c, pa, pb);
      };
      Dq1Cursor c0 = first, c1 = first;
      dq1_next(p, resp_tokens, c1);
      Dq1Cursor c2 = c1;
      dq1_next(p, resp_tokens, c2);
      int pa0, pb0, pa1, pb1;
      pages_of(c0, pa0, pb0);
      pages_of(c1, pa1, pb1);
      // chunk order = consumption order: S(0) T(0) [S(i+1) ACC(i) T(i+1)] ...; ACC re-reads K
      load_op(0, c0, pa0, pb0);
      load_op(1, c0, pa0, pb0);
      for (int i = 0; i < n_tiles; ++i) {
        int pa2, pb2;
        pages_of(c2, pa2, pb2);
        if (i + 1 < n_tiles) load_op(0, c1, pa1, pb1);
        load_op(0, c0, pa0, pb0);
        if (i + 1 < n_tiles) load_op(1, c1, pa1, pb1);
        c0 = c1; c1 = c2;
        dq1_next(p, resp_tokens, c2);
        pa0 = pa1; pb0 = pb1; pa1 = pa2; pb1 = pb2;
      }
      LS_D1DUMP(0, tw0);
      LS_D1DUMP(1, clock64() - t_kernel0);
      LS_D1DUMP(2, (long long)n_tiles);
      if (*abort_flag) {   // aborted: wait (bounded) for the copies already started
        for (uint32_t s2 = 0; s2 < nring && s2 < issued; ++s2) {
          const uint32_t last = ((issued - 1 - s2) / nring) * nring + s2;
          const uint64_t t_start = globaltimer_ns();
          while (!mbar_try_wait(&full[s2], (last / nring) & 1, 1000) && globaltimer_ns() - t_start < 100000000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // =========================================================== MMA issuer (one thread)
    if (lane == 0 && n_tiles > 0) {
      constexpr uint32_t idesc_st = make_idesc(128, 128, 0, 0);
      constexpr uint32_t idesc_acc = make_idesc(128, 128, 0, 1);
      constexpr uint32_t hi = sdesc_hi(1024);
      const uint32_t a1_lo = sdesc_lo(smem_u32(a1_smem), 16), a2_lo = sdesc_lo(smem_u32(a2_smem), 16);
      const uint32_t ring_k_lo = sdesc_lo(smem_u32(ring), 16);       // K-major view of a chunk
      const uint32_t ring_m_lo = sdesc_lo(smem_u32(ring), 16384);    // MN-major view: 16 KB group pitch
      uint32_t slot = 0, phase = 0;
      bool ok = mbar_wait(a_full, 0, abort_flag);
      auto advance = [&]() {
        if (++slot == nring) { slot = 0; phase ^= 1; }
      };
      auto issue_op = [&](int op) {       // S = Q K^T (0) or T = dO V^T (1)
        const uint32_t a_lo = op == 0 ? a1_lo : a2_lo;
        const uint32_t d = op == 0 ? tmem_s : tmem_t;
#pragma unroll
        for (int c = 0; c < C::NC; ++c) {
          ok = ok && LS_BTWAIT(tw0, mbar_wait(&full[slot], phase, abort_flag));
          if (!ok) return;
          tc_fence_after();
          const uint32_t b_lo = ring_k_lo + slot * (kBwdChunk >> 4);
#pragma unroll
          for (int s2 = 0; s2 < 2; ++s2)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              mma_ss(d, sdesc(a_lo + (((2 * c + s2) * slab + k * 32) >> 4), hi),
                     sdesc(b_lo + ((s2 * 16384 + k * 32) >> 4), hi), idesc_st, (c | s2 | k) != 0);
          mma_commit(&empty[slot]);
          advance();
        }
        mma_commit(op == 0 ? s_full : t_full);
      };
      auto issue_acc = [&](int i) {
        uint32_t cs[C::NC], cph[C::NC];
#pragma unroll
        for (int c = 0; c < C::NC; ++c) {
          cs[c] = slot;
          cph[c] = phase;
          advance();
        }
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) {
          ok = ok && LS_BTWAIT(tw1, mbar_wait(&e_full[qd], i & 1, abort_flag));
          if (!ok) return;
          tc_fence_after();
#pragma unroll
          for (int c = 0; c < C::NC; ++c) {
            if (qd == 0) {
              ok = ok && LS_BTWAIT(tw2, mbar_wait(&full[cs[c]], cph[c], abort_flag));
              if (!ok) return;
              tc_fence_after();
            }
            const uint32_t b_lo = ring_m_lo + cs[c] * (kBwdChunk >> 4);
#pragma unroll
            for (int kk = 0; kk < 2; ++kk)
              mma_ts(tmem_acc + c * 128, tmem_t + (2 * qd + kk) * 8, sdesc(b_lo + (((2 * qd + kk) * 2048) >> 4), hi),
                     idesc_acc, (i | qd | kk) != 0);
            if (qd == 3) mma_commit(&empty[cs[c]]);
          }
        }
        if (i == n_tiles - 1) mma_commit(acc_final);
      };
      if (ok) issue_op(0);
      if (ok) issue_op(1);
      for (int i = 0; i < n_tiles && ok; ++i) {
        if (i + 1 < n_tiles) {
          ok = ok && LS_BTWAIT(tw3, mbar_wait(s_read, i & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
          issue_op(0);
        }
        if (ok) issue_acc(i);
        if (ok && i + 1 < n_tiles) issue_op(1);
      }
      LS_D1DUMP(8, tw0);
      LS_D1DUMP(9, tw1);
      LS_D1DUMP(10, tw2);
      LS_D1DUMP(11, tw3);
      LS_D1DUMP(12, clock64() - t_kernel0);
    }
  } else {
    // =========================================================== elementwise + epilogue
    const int quad = warp & 3;
    const int sub = (warp - 2) >> 2;                       // four threads per row: thread `sub` owns the 32-key quarter `sub`
    const int row = quad * 32 + lane;
    const int hj = row / p.bt;                            // head and token of this row of the tile
    const int r_tok = t0 + row - hj * p.bt;
    const bool row_ok = hj < p.bh && r_tok < p.R && h + hj < (kvh + 1) * p.g;
    const int r_idx = min(r_tok, p.R - 1);
    const int hr = min(h + hj, p.Hq - 1);
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    const size_t ri = (size_t)r_idx * p.Hq + hr;
    bool ok = true;
    if (n_tiles > 0) {
      const float lse2_row = p.lse[ri] * kLog2e;
      const float delta_row = p.delta[ri];
      Dq1Cursor cu = first;
      for (int i = 0; i < n_tiles; ++i) {
        const int64_t lim = cu.is_resp ? (int64_t)r_idx : cu.tokens - 1;
        const int64_t key0 = (int64_t)cu.i * 128;
        const bool edge = __any_sync(0xffffffffu, key0 + 127 > lim);
        // No thread leaves this loop on its own: a wait that gave up is remembered in `ok` and put
        // to the vote at the tile's named barrier, where all 512 leave together.
        ok = ok && LS_BTWAIT(tw0, mbar_wait(s_full, i & 1, abort_flag));
        tc_fence_after();
        uint32_t sr[32];
        tmem_ld32(tmem_s + lane_sel + 32 * sub, sr);
        tc_wait_ld32(sr);
        tc_fence_before();
        mbar_arrive(s_read);                 // S is in registers: the next tile's S may overwrite the buffer
        float pr[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          float e = ex2(fmaf(__uint_as_float(sr[j]), p.scale_log2, -lse2_row));
          if (edge && key0 + 32 * sub + j > lim) e = 0.f;
          pr[j] = e;
        }
        ok = ok && LS_BTWAIT(tw1, mbar_wait(t_full, i & 1, abort_flag));
        tc_fence_after();
        uint32_t tr[32];
        tmem_ld32(tmem_t + lane_sel + 32 * sub, tr);
        tc_wait_ld32(tr);
        // E (bf16) goes over T's columns, which the row's other threads read too: every T read of the
        // CTA comes before any E write (named barrier 1, which also carries the vote)
        ok = LS_BTWAIT(tw2, bar_and(1, 512, ok));
        if (!ok) break;
        uint32_t pk[16];
#pragma unroll
        for (int j = 0; j < 32; j += 2)
          pk[j >> 1] = pack_bf16(pr[j] * (__uint_as_float(tr[j]) - delta_row),
                                 pr[j + 1] * (__uint_as_float(tr[j + 1]) - delta_row));
        tmem_st16(tmem_t + lane_sel + 16 * sub, pk);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(&e_full[sub]);
        dq1_next(p, resp_tokens, cu);
      }
      if (threadIdx.x == 64) {
        LS_D1DUMP(16, tw0);
        LS_D1DUMP(17, tw1);
        LS_D1DUMP(18, tw2);
        LS_D1DUMP(19, clock64() - t_kernel0);
      }
      ok = __all_sync(0xffffffffu, ok);
      if (ok) ok = bwd_wait_warp(acc_final, 0, abort_flag);
      if (ok) tc_fence_after();
    }
    // ---- epilogue: the range's sum goes to its own partial (one tile per KV group), or the link's sum is
    // added to the running dQ of the tile's rows, in link order
    if (p.dq_split) {
      if (ok)
        dq_store_row<D / 4>(tmem_acc + lane_sel + sub * (D / 4), n_tiles > 0, false, false, p.scale,
                            p.dq_split + ((size_t)range * p.R * p.Hq + ri) * D + sub * (D / 4), nullptr, row_ok);
    } else {
      const bool fold = it.link > 0, last = it.link == p.parts;
      int* counter = p.ctl + kChainHeaderInts + kvh * p.nq_tiles + qtile;
      if (ok && fold) ok = __all_sync(0xffffffffu, chain_wait(counter, it.link, p.ctl, abort_flag));
      if (ok)
        dq_store_row<D / 4>(tmem_acc + lane_sel + sub * (D / 4), n_tiles > 0, fold, last, p.scale,
                            p.dq_acc + ri * D + sub * (D / 4), p.dq + ri * D + sub * (D / 4), row_ok);
      const bool all_ok = bar_and(2, 512, ok);     // every row of the tile is written
      if (row == 0 && sub == 0 && all_ok) chain_publish(counter, it.link + 1);
    }
  }
#undef LS_D1DUMP

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
  if (threadIdx.x == 0 && *abort_flag) {
    if (p.status) atomicExch(p.status, (int)LS_ERR_TIMEOUT);
    st_relaxed_gpu(p.ctl + 1, 1);    // ends every other chain wait of this launch
  }
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

void launch_delta(const void* d_o, const float* o_f32, int64_t rows, int dv, float* delta, cudaStream_t st) {
  delta_kernel<<<(int)((rows + 7) / 8), 256, 0, st>>>(static_cast<const __nv_bfloat16*>(d_o), o_f32, rows, dv, delta);
}

template <int D, int MODE>
static ls_status_t launch_kv(const BwdParams& prm, int grid, cudaStream_t st, bool timed) {
  using C = BwdCfg<D>;
  static bool configured[64] = {};
  const ls_status_t cs = configure_smem(bwd_kv_kernel<D, MODE>, C::SMEM_BYTES, configured);
  if (cs != LS_OK) return cs;
  constexpr int which = MODE == MODE_DK ? LS_KERNEL_BWD_DK : LS_KERNEL_BWD_DV;
  if (timed) profile_begin(which, st);
  bwd_kv_kernel<D, MODE><<<grid, kBwdThreads, C::SMEM_BYTES, st>>>(prm);
  if (timed) profile_end(which, st);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

// ---------------------------------------------------------------------------------
// dQ pass on CTA pairs with 256-key tiles (D = 256).  With N = 256 every MMA runs at the math
// rate (the resident operand is re-read from shared memory half as often per key).  TMEM has
// room for the accumulator and ONE 256-column score buffer, so a tile goes S -> p (kept in
// registers, 128 per thread, two threads per row) -> T into the same buffer -> E = p (T - Delta)
// in four 64-key quarters -> dQ += E K per quarter.
// Chunks of 16 KB per CTA: K or V as (this CTA's 128 keys x 64 channels) for S / T, and K as
// (64 keys x this CTA's 128 channels) for the accumulate.
// ---------------------------------------------------------------------------------
constexpr int kDq3Tpr = 4;                              // threads per row of the elementwise warps
constexpr int kDq3Threads = 64 + 128 * kDq3Tpr;         // producer warp, MMA warp, 4 * kDq3Tpr elementwise warps
constexpr int kDq3Cw = 64 / kDq3Tpr;                    // columns of every 64-key quarter one thread owns

struct Dq3Cfg {
  static constexpr int D = 256;
  static constexpr int SLABS = 4;
  static constexpr int RING = 6;
  static constexpr int A_BYTES = 2 * SLABS * 16384;
  static constexpr int SMEM_BYTES = 1024 + A_BYTES + RING * kDq2Chunk + 512;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kDq3Threads, 1)
    bwd_dq3_kernel(const __grid_constant__ BwdParams p) {
  using C = Dq3Cfg;
  constexpr int D = 256;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* a1_smem = smem;
  uint8_t* a2_smem = smem + C::SLABS * 16384;
  uint8_t* ring = smem + C::A_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + C::RING * kDq2Chunk);
  uint64_t* a_full = bars;               // (even CTA) both CTAs' resident operands landed
  uint64_t* full = bars + 1;             // (even CTA) both halves of a chunk landed
  uint64_t* empty = full + C::RING;      // (each CTA) chunk consumed
  uint64_t* s_full = empty + C::RING;    // (each CTA) S in TMEM
  uint64_t* s_read = s_full + 1;         // (even CTA) every row thread of both CTAs has pulled S: one arrival per warp
  uint64_t* t_full = s_read + 1;         // (each CTA) T in TMEM
  uint64_t* e_full = t_full + 1;         // [4] (even CTA) quarter of E in both CTAs' TMEM: one arrival per warp
  uint64_t* acc_final = e_full + 4;      // (each CTA)
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_final + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  int* work_idx = const_cast<int*>(abort_flag) + 1;   // (even CTA) the pair's work item

  long long tw0 = 0, tw1 = 0, tw2 = 0;
  (void)tw0; (void)tw1; (void)tw2;
  const long long t_kernel0 = clock64();
  (void)t_kernel0;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    mbar_init(a_full, 1);
    for (int i = 0; i < C::RING; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    mbar_init(s_full, 1);
    mbar_init(s_read, 8 * kDq3Tpr);
    mbar_init(t_full, 1);
    for (int i = 0; i < 4; ++i) mbar_init(&e_full[i], 8 * kDq3Tpr);
    mbar_init(acc_final, 1);
    *abort_flag = 0;
    // work items are handed out in launch order of the pairs that ask (see chain_wait)
    if (leader) *work_idx = atomicAdd(p.ctl, 1);
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_holder, 512);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  const uint32_t tmem_acc = tmem_base;
  const uint32_t tmem_st = tmem_base + D;      // S, then T, then E (bf16) over its first 128 columns

  const int npairs = (p.nq_tiles + 1) / 2;
  const DqItem it = dq_item(p, (int)ld_shared_cluster_u32(mapa_u32(smem_u32(work_idx), 0)), npairs);
  const int pairi = it.pairi, part = it.part, kvh = it.kvh;
  const bool is_resp = it.is_resp;
  auto tile_of = [&](int qt, int& hh, int& r0) {
    if (qt < p.nq_tiles) {
      hh = kvh * p.g + (qt / p.tiles_tok) * p.bh;     // tile of bt tokens x bh heads (RowTiling)
      r0 = (qt % p.tiles_tok) * p.bt;
    } else {                                           // odd tile count: the pair's second CTA works on zero rows
      hh = kvh * p.g + p.g - 1;
      r0 = p.tiles_tok * p.bt;
    }
  };
  const int qtile = 2 * pairi + (int)rank;
  int h, row0, h_o, row0_o;
  tile_of(qtile, h, row0);
  tile_of(2 * pairi + 1 - (int)rank, h_o, row0_o);
  int64_t tokens;
  int page_off = 0, n_pages = 0, tail_slot = -1;
  if (is_resp) {
    tokens = p.no_resp ? 0 : min(p.R, max(row0, row0_o) + p.bt);
  } else {
    tokens = p.part_tokens[part];
    page_off = p.part_page_offset[part];
    n_pages = p.part_page_offset[part + 1] - page_off;
    tail_slot = p.part_tail_slot[part];
  }
  const int n_tiles = (int)((tokens + 255) / 256);

  if (warp == 0) {
    // =========================================================== producer (one thread per CTA)
    if (lane == 0 && n_tiles > 0) {
      const int a_rows = p.bt * p.bh;
      if (leader) mbar_arrive_expect_tx(a_full, 2 * 2 * C::SLABS * a_rows * 128);
      for (int c = 0; c < C::SLABS; ++c) {
        tma_load_5d_pair(a1_smem + c * 16384, &p.a1_map, a_full, 0, row0, c, h, 0);
        tma_load_5d_pair(a2_smem + c * 16384, &p.a2_map, a_full, 0, row0, c, h, 0);
      }
      const int32_t* pages = p.part_pages + page_off;
      const int pg_mask = (1 << p.pg_shift) - 1;
      const bool small_pages = !is_resp && p.pg_shift == 6;
      auto page_at = [&](int tok) -> int {       // physical page holding key `tok` of this partial
        if (is_resp) return 0;
        const int ps = tok >> p.pg_shift;
        return (ps < n_pages) ? __ldg(pages + ps) : p.num_phys_pages;   // past the end: TMA fills zeros
      };
      uint32_t slot = 0, phase = 0, issued = 0;
      bool ok = true;
      auto acquire = [&]() -> uint8_t* {
        ok = ok && LS_BTWAIT(tw0, mbar_wait(&empty[slot], phase ^ 1, abort_flag));
        if (ok && leader) mbar_arrive_expect_tx(&full[slot], 2 * kDq2Chunk);
        return ring + slot * kDq2Chunk;
      };
      auto advance = [&]() {
        ++issued;
        if (++slot == (uint32_t)C::RING) { slot = 0; phase ^= 1; }
      };
      // pq[j]: page of keys [256 i + 64 j, +64) of the tile being loaded
      auto load_tile = [&](int i, const int* pq) {
        const int tk = i * 256 + (int)rank * 128;          // this CTA's 128 keys for S and T
        for (int which = 0; which < 2; ++which) {
          for (int g = 0; g < 4; ++g) {
            uint8_t* dst = acquire();
            if (ok) {
              if (is_resp) {
                tma_load_5d_pair(dst, which ? &p.rv_m : &p.rk_m, &full[slot], 0, tk, g, kvh, 0);
              } else if (!small_pages) {
                const bool tail = (tk >> p.pg_shift) == tail_slot;
                const CUtensorMap* m = which ? (tail ? &p.pv_m_tail : &p.pv_m) : (tail ? &p.pk_m_tail : &p.pk_m);
                tma_load_5d_pair(dst, m, &full[slot], 0, tk & pg_mask, g, kvh, pq[2 * rank]);
              } else {
                const int sa = tk >> 6;
                const CUtensorMap* ma = which ? (sa == tail_slot ? &p.pv_m_tail : &p.pv_m)
                                              : (sa == tail_slot ? &p.pk_m_tail : &p.pk_m);
                const CUtensorMap* mb = which ? (sa + 1 == tail_slot ? &p.pv_m_tail : &p.pv_m)
                                              : (sa + 1 == tail_slot ? &p.pk_m_tail : &p.pk_m);
                tma_load_5d_pair(dst, ma, &full[slot], 0, 0, g, kvh, pq[2 * rank]);
                tma_load_5d_pair(dst + 8192, mb, &full[slot], 0, 0, g, kvh, pq[2 * rank + 1]);
              }
            }
            advance();
          }
        }
        for (int j = 0; j < 4; ++j) {                       // K for the accumulate: 64 keys x this CTA's 128 channels
          uint8_t* dst = acquire();
          if (ok) {
            const int tq = i * 256 + j * 64;
            if (is_resp) {
              tma_load_5d_pair(dst, &p.rk_s, &full[slot], 0, tq, 2 * (int)rank, kvh, 0);
            } else {
              const bool tail = (tq >> p.pg_shift) == tail_slot;
              tma_load_5d_pair(dst, tail ? &p.pk_s_tail : &p.pk_s, &full[slot], 0, tq & pg_mask, 2 * (int)rank, kvh,
                               pq[j]);
            }
          }
          advance();
        }
      };
      int pq0[4], pq1[4];
      for (int j = 0; j < 4; ++j) pq0[j] = page_at(j * 64);
      for (int i = 0; i < n_tiles; ++i) {
        for (int j = 0; j < 4; ++j) pq1[j] = (i + 1 < n_tiles) ? page_at((i + 1) * 256 + j * 64) : 0;   // next tile
        load_tile(i, pq0);
        for (int j = 0; j < 4; ++j) pq0[j] = pq1[j];
      }
      LS_BTDUMP(0, tw0);
      LS_BTDUMP(1, clock64() - t_kernel0);
      if (*abort_flag && leader) {
        for (uint32_t s2 = 0; s2 < (uint32_t)C::RING && s2 < issued; ++s2) {
          const uint32_t last = ((issued - 1 - s2) / C::RING) * C::RING + s2;
          const uint64_t t_start = globaltimer_ns();
          while (!mbar_try_wait(&full[s2], (last / C::RING) & 1, 1000) && globaltimer_ns() - t_start < 100000000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // =========================================================== MMA issuer (one thread of the even CTA)
    if (leader && lane == 0 && n_tiles > 0) {
      constexpr uint32_t idesc_st = make_idesc(256, 256, 0, 0);
      constexpr uint32_t idesc_acc = make_idesc(256, 256, 0, 1);
      constexpr uint32_t hi = sdesc_hi(1024);
      const uint32_t a1_lo = sdesc_lo(smem_u32(a1_smem), 16), a2_lo = sdesc_lo(smem_u32(a2_smem), 16);
      const uint32_t ring_k_lo = sdesc_lo(smem_u32(ring), 16);       // K-major 128 keys x 64 channels
      const uint32_t ring_m_lo = sdesc_lo(smem_u32(ring), 8192);     // MN-major 64 keys x 2 groups of 64 channels
      uint32_t slot = 0, phase = 0;
      bool ok = mbar_wait(a_full, 0, abort_flag);
      auto advance = [&]() {
        if (++slot == (uint32_t)C::RING) { slot = 0; phase ^= 1; }
      };
      for (int i = 0; i < n_tiles && ok; ++i) {
#pragma unroll
        for (int op = 0; op < 2; ++op) {
          if (op == 1) {                     // T overwrites S: every row thread must have pulled its S first
            ok = ok && LS_BTWAIT(tw1, mbar_wait(s_read, i & 1, abort_flag));
            if (!ok) break;
            tc_fence_after();
          }
          const uint32_t a_lo = op == 0 ? a1_lo : a2_lo;
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            ok = ok && LS_BTWAIT(tw0, mbar_wait(&full[slot], phase, abort_flag));
            if (!ok) break;
            tc_fence_after();
            const uint32_t b_lo = ring_k_lo + slot * (kDq2Chunk >> 4);
#pragma unroll
            for (int k = 0; k < 4; ++k)
              mma_ss_pair(tmem_st, sdesc(a_lo + ((g * 16384 + k * 32) >> 4), hi), sdesc(b_lo + ((k * 32) >> 4), hi),
                          idesc_st, (g | k) != 0);
            mma_commit_pair(&empty[slot]);
            advance();
          }
          if (!ok) break;
          mma_commit_pair(op == 0 ? s_full : t_full);
        }
        if (!ok) break;
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) {
          ok = ok && LS_BTWAIT(tw2, mbar_wait(&e_full[qd], i & 1, abort_flag));
          ok = ok && LS_BTWAIT(tw0, mbar_wait(&full[slot], phase, abort_flag));
          if (!ok) break;
          tc_fence_after();
          const uint32_t b_lo = ring_m_lo + slot * (kDq2Chunk >> 4);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            mma_ts_pair(tmem_acc, tmem_st + (4 * qd + kk) * 8, sdesc(b_lo + ((kk * 2048) >> 4), hi), idesc_acc,
                        (i | qd | kk) != 0);
          mma_commit_pair(&empty[slot]);
          advance();
        }
        if (ok && i == n_tiles - 1) mma_commit_pair(acc_final);
      }
      LS_BTDUMP(8, tw0);
      LS_BTDUMP(9, tw1);
      LS_BTDUMP(10, tw2);
      LS_BTDUMP(11, clock64() - t_kernel0);
    }
  } else {
    // =========================================================== elementwise + epilogue (both CTAs)
    const int quad = warp & 3;
    const int sub = (warp - 2) >> 2;                // which kDq3Cw columns of every 64-key quarter this thread owns
    constexpr int CW = kDq3Cw;
    constexpr int NT = 128 * kDq3Tpr;               // elementwise threads of the CTA
    const int row = quad * 32 + lane;
    const int hj = row / p.bt;                      // head and token of this row of the tile
    const int r_idx = row0 + row - hj * p.bt;
    const int hr = min(h + hj, p.Hq - 1);
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    const bool tile_ok = qtile < p.nq_tiles;
    const bool row_ok = tile_ok && hj < p.bh && r_idx < p.R && h + hj < (kvh + 1) * p.g;
    const size_t ri = (size_t)min(r_idx, p.R - 1) * p.Hq + hr;
    bool ok = true;
    if (n_tiles > 0) {
      const float lse2_row = p.lse[ri] * kLog2e;
      const float delta_row = p.delta[ri];
      const int64_t lim = is_resp ? (int64_t)min(r_idx, p.R - 1) : tokens - 1;
      const uint32_t s_read_remote = mapa_u32(smem_u32(s_read), 0);
      uint32_t e_remote[4];
#pragma unroll
      for (int qd = 0; qd < 4; ++qd) e_remote[qd] = mapa_u32(smem_u32(&e_full[qd]), 0);
      for (int i = 0; i < n_tiles; ++i) {
        const int key0 = i * 256;
        const bool edge = __any_sync(0xffffffffu, (int64_t)key0 + 255 > lim);
        // No thread leaves this loop on its own: a wait that gave up is remembered in `ok` and put
        // to the vote at the first named barrier of the tile, where all leave together.
        ok = ok && LS_BTWAIT(tw0, mbar_wait(s_full, i & 1, abort_flag));
        tc_fence_after();
        // p = exp(s - LSE) for this thread's 4 x CW columns: all four TMEM loads in flight at once,
        // p kept as packed bf16 pairs until T is ready
        uint32_t sr[4 * CW];
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) tmem_ld16(tmem_st + lane_sel + 64 * qd + CW * sub, sr + CW * qd);
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) tc_wait_ld16(sr + CW * qd);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(s_read_remote);    // this warp no longer needs S: T may overwrite it
        uint32_t pp[2 * CW];
#pragma unroll
        for (int j = 0; j < 4 * CW; j += 2) {
          float e0 = ex2(fmaf(__uint_as_float(sr[j]), p.scale_log2, -lse2_row));
          float e1 = ex2(fmaf(__uint_as_float(sr[j + 1]), p.scale_log2, -lse2_row));
          if (edge) {
            const int64_t col = (int64_t)key0 + 64 * (j / CW) + CW * sub + (j % CW);
            if (col > lim) e0 = 0.f;
            if (col + 1 > lim) e1 = 0.f;
          }
          pp[j >> 1] = pack_bf16(e0, e1);
        }
        ok = ok && LS_BTWAIT(tw1, mbar_wait(t_full, i & 1, abort_flag));
        tc_fence_after();
        uint32_t tr[2][CW];
        tmem_ld16(tmem_st + lane_sel + CW * sub, tr[0]);
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) {
          tc_wait_ld16(tr[qd & 1]);
          if (qd < 3) tmem_ld16(tmem_st + lane_sel + 64 * (qd + 1) + CW * sub, tr[(qd + 1) & 1]);   // in flight meanwhile
          uint32_t pk[CW / 2];
#pragma unroll
          for (int j = 0; j < CW; j += 2) {
            const uint32_t pw = pp[(CW / 2) * qd + (j >> 1)];
            pk[j >> 1] = pack_bf16(__uint_as_float(pw << 16) * (__uint_as_float(tr[qd & 1][j]) - delta_row),
                                   __uint_as_float(pw & 0xffff0000u) * (__uint_as_float(tr[qd & 1][j + 1]) - delta_row));
          }
          // E (bf16 pairs) of quarter q goes to columns [32 q, 32 q + 32) of the buffer: T columns that
          // this quarter or an earlier one has read -- by any thread of the row, hence the barrier
          if (qd == 0) {
            ok = bar_and(1, NT, ok);
            if (!ok) break;
          } else {
            bar_sync(1, NT);
          }
          tmem_st8(tmem_st + lane_sel + 32 * qd + (CW / 2) * sub, pk);
          tc_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(e_remote[qd]);
        }
        if (!ok) break;          // (uniform: decided by the vote above)
      }
      if (threadIdx.x == 64) {
        LS_BTDUMP(16, tw0);
        LS_BTDUMP(17, tw1);
        LS_BTDUMP(18, clock64() - t_kernel0);
      }
      if (ok) ok = bwd_wait_warp(acc_final, 0, abort_flag);
      if (ok) tc_fence_after();
    }
    // ---- epilogue: add this part's sum to the running dQ of the row tile, in link order
    const bool fold = it.link > 0, last = it.link == p.parts;
    int* counter = p.ctl + kChainHeaderInts + kvh * p.nq_tiles + min(qtile, p.nq_tiles - 1);
    if (tile_ok) {
      if (ok && fold) ok = __all_sync(0xffffffffu, chain_wait(counter, it.link, p.ctl, abort_flag));
      if (ok)
        dq_store_row<D / kDq3Tpr>(tmem_acc + lane_sel + sub * (D / kDq3Tpr), n_tiles > 0, fold, last, p.scale,
                                  p.dq_acc + ri * D + sub * (D / kDq3Tpr), p.dq + ri * D + sub * (D / kDq3Tpr), row_ok);
      const bool all_ok = bar_and(2, 128 * kDq3Tpr, ok);     // every row of the tile is written
      if (row == 0 && sub == 0 && all_ok) chain_publish(counter, it.link + 1);
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 512);
  }
  if (threadIdx.x == 0 && *abort_flag) {
    if (p.status) atomicExch(p.status, (int)LS_ERR_TIMEOUT);
    st_relaxed_gpu(p.ctl + 1, 1);    // ends every other chain wait of this launch
  }
}

// Shared memory of the single-CTA dQ kernel: alignment slack, Q and dO rows of the tile, the ring, barriers.
constexpr int kDq1SmemMax = 232448;     // 227 KB
constexpr int kDq1RingMax = 8;
template <int D>
static ls_status_t launch_dq1(BwdParams& prm, int64_t grid, cudaStream_t st) {
  using C = BwdCfg<D>;
  static bool configured[64] = {};
  if (grid > INT32_MAX) return LS_ERR_UNSUPPORTED_SHAPE;
  const int rows_pad = std::min(128, (prm.bt * prm.bh + 7) / 8 * 8);
  prm.a_slab_bytes = rows_pad * 128;
  const int a_bytes = 2 * C::SLABS * prm.a_slab_bytes;
  prm.dq1_ring = std::min(kDq1RingMax, (kDq1SmemMax - 1024 - 512 - a_bytes) / kBwdChunk);
  const int smem_bytes = 1024 + a_bytes + prm.dq1_ring * kBwdChunk + 512;
  const ls_status_t cs = configure_smem(bwd_dq1_kernel<D>, kDq1SmemMax, configured);
  if (cs != LS_OK) return cs;
  profile_begin(LS_KERNEL_BWD_DQ, st);
  bwd_dq1_kernel<D><<<(int)grid, kDq1Threads, smem_bytes, st>>>(prm);
  profile_end(LS_KERNEL_BWD_DQ, st);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

static ls_status_t launch_dq3(const BwdParams& prm, int64_t grid, cudaStream_t st) {
  static bool configured[64] = {};
  if (grid > INT32_MAX) return LS_ERR_UNSUPPORTED_SHAPE;
  const ls_status_t cs = configure_smem(bwd_dq3_kernel, Dq3Cfg::SMEM_BYTES, configured);
  if (cs != LS_OK) return cs;
  profile_begin(LS_KERNEL_BWD_DQ, st);
  bwd_dq3_kernel<<<(int)grid, kDq3Threads, Dq3Cfg::SMEM_BYTES, st>>>(prm);
  profile_end(LS_KERNEL_BWD_DQ, st);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

template <int D>
static ls_status_t launch_dq2(const BwdParams& prm, int64_t grid, cudaStream_t st) {
  using C = Dq2Cfg<D>;
  static bool configured[64] = {};
  if (grid > INT32_MAX) return LS_ERR_UNSUPPORTED_SHAPE;
  const ls_status_t cs = configure_smem(bwd_dq2_kernel<D>, C::SMEM_BYTES, configured);
  if (cs != LS_OK) return cs;
  profile_begin(LS_KERNEL_BWD_DQ, st);
  bwd_dq2_kernel<D><<<(int)grid, kBwdThreads, C::SMEM_BYTES, st>>>(prm);
  profile_end(LS_KERNEL_BWD_DQ, st);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

}  // namespace ls

extern "C" ls_status_t ls_replay_attn_bwd(const ls_pages_t* h, const ls_attn_params_t* prm, const void* q,
                                          const void* k_resp, const void* v_resp, const float* o_f32,
                                          const float* lse, const void* d_o, void* dq, void* dk_resp,
                                          void* dv_resp, void* workspace, size_t workspace_bytes,
                                          int32_t* status_dev, void* stream) {
  ls_status_t st = ls::check_handle(h, prm);
  if (st != LS_OK) return st;
  const bool no_resp = (prm->flags & LS_FLAG_NO_RESPONSE_BLOCK) != 0;
  if (!q || !o_f32 || !lse || !d_o || !dq) return LS_ERR_INVALID_ARG;
  if (!no_resp && (!k_resp || !v_resp || !dk_resp || !dv_resp)) return LS_ERR_INVALID_ARG;
  if (no_resp) k_resp = v_resp = q;                    // response maps are encoded but never used
  const ls_pages_desc_t& d = h->desc;
  if (prm->R < 1 || prm->num_q_heads < 1 || prm->num_q_heads % d.num_kv_heads != 0) return LS_ERR_INVALID_ARG;
  if (!(prm->scale > 0.f)) return LS_ERR_INVALID_ARG;
  const bool mla = d.dim_k == 576 && d.dim_v == 512;
  const void* ptrs[] = {q, k_resp, v_resp, o_f32, d_o, dq, dk_resp, dv_resp, workspace};
  for (const void* ptr : ptrs)
    if (!ls::aligned16(ptr)) return LS_ERR_ALIGNMENT;
  const size_t need = ls_replay_attn_workspace_bytes(h, prm, LS_WORKSPACE_BWD);
  if (!workspace || workspace_bytes < need) return LS_ERR_WORKSPACE;
  const bool add_grad = (prm->flags & LS_FLAG_ADD_SUFFIX_GRAD) != 0;
  if ((add_grad || !h->suffix_blocks.empty()) && (mla || !h->dk_grad)) return LS_ERR_INVALID_ARG;

  const int R = prm->R, Hq = prm->num_q_heads, Hkv = d.num_kv_heads, D = d.dim_k;
  const int g = Hq / Hkv;
  const int tiles_per_head = (R + 127) / 128;
  const int64_t rows = (int64_t)R * Hq;
  // workspace: Delta | hand-over control words | fp32 running dQ (one per partial for the generic 576/512 path)
  float* delta = static_cast<float*>(workspace);
  const size_t delta_bytes = ((size_t)rows * sizeof(float) + 15) & ~(size_t)15;
  int* ctl = reinterpret_cast<int*>(static_cast<char*>(workspace) + delta_bytes);
  int64_t chains = (int64_t)Hkv * g * tiles_per_head;
  if (mla && ls::mla_dq_fast(h)) chains = std::max(chains, ls::mla_dq_blocks(h, R, Hq));
  const size_t ctl_bytes = ((size_t)(ls::kChainHeaderInts + chains) * sizeof(int) + 15) & ~(size_t)15;
  float* kv_scratch = reinterpret_cast<float*>(reinterpret_cast<char*>(ctl) + ctl_bytes);   // 576/512 only
  const int kv_hsplit = mla ? ls::mla_kv_hsplit(h, R, Hq) : 1;
  float* dq_acc = kv_scratch + (kv_hsplit > 1 ? (size_t)kv_hsplit * R * Hkv * D : 0);
  if (kv_hsplit == 1) kv_scratch = nullptr;
  const int parts = h->num_parts();
  cudaStream_t cs = static_cast<cudaStream_t>(stream);

  ls::launch_delta(d_o, o_f32, rows, d.dim_v, delta, cs);

  if (mla) {
    const bool mla_fast = ls::mla_dq_fast(h);
    if (no_resp) {       // prefix parts only: the transposed kernel walks them all and writes dQ
      if (!mla_fast) return LS_ERR_UNSUPPORTED_SHAPE;
      // (no response partial: the first fp32 region is the running dQ of a chained launch, the split
      // partials follow it)
      return ls::bwd_mla_dq(h, prm, q, d_o, lse, delta, nullptr,
                            ls::mla_dq_split(h, R, Hq).chain ? dq_acc : dq_acc + rows * D, ctl, dq, status_dev, cs);
    }
    ls_status_t ms =
        ls::bwd_mla(h, prm, q, k_resp, v_resp, lse, delta, d_o, dq_acc, dk_resp, dv_resp, mla_fast, kv_scratch, status_dev, cs);
    if (ms != LS_OK) return ms;
    if (mla_fast) return ls::bwd_mla_dq(h, prm, q, d_o, lse, delta, dq_acc, dq_acc + rows * D, ctl, dq, status_dev, cs);
    const int64_t n4m = rows * D / 4;
    ls::dq_reduce_kernel<<<(int)std::min<int64_t>((n4m + 255) / 256, 148 * 16), 256, 0, cs>>>(
        dq_acc, parts + 1, n4m, prm->scale, static_cast<__nv_bfloat16*>(dq));
    return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
  }

  auto dense_map = [&](CUtensorMap* m, const void* base, int heads, int box_tok, int groups) {
    return ls::encode_map5(m, base, D, R, heads, 1, (int64_t)heads * D, D, (int64_t)R * heads * D, box_tok, groups);
  };
  const bool small_pages = d.page_size == 64;
  const int mbox = small_pages ? 64 : 128;
  ls::BwdParams P;
  P.part_pages = h->d_part_pages;
  P.part_page_offset = h->d_part_page_offset;
  P.part_tail_slot = h->d_part_tail_slot;
  P.part_tokens = h->d_part_tokens;
  P.lse = lse;
  P.delta = delta;
  P.dq_acc = dq_acc;
  P.dq_split = nullptr;
  P.dq = static_cast<__nv_bfloat16*>(dq);
  P.ctl = ctl;
  P.out = nullptr;
  P.grad = nullptr;
  P.status = status_dev;
  P.timing = ls::g_timing_buffer;
  P.R = R;
  P.Hq = Hq;
  P.Hkv = Hkv;
  P.g = g;
  P.parts = parts;
  P.pg_shift = ls::pg_shift_of(d.page_size);
  P.tiles_per_head = tiles_per_head;
  P.nq_tiles = g * tiles_per_head;
  P.num_phys_pages = (int)std::min<int64_t>(d.num_phys_pages, INT32_MAX);
  P.keys_paged = P.key_page_off = P.key_tokens = P.grad_slot0 = 0;
  P.scale = prm->scale;
  P.scale_log2 = prm->scale * ls::kLog2e;

  // ---- dQ: rows = queries, columns = keys of every part, summed through the running dQ
  P.no_resp = no_resp ? 1 : 0;
  const ls::RowTiling rt = ls::row_tiling(R, g, 128);
  P.bt = rt.bt;
  P.bh = rt.bh;
  P.tiles_tok = rt.tiles_tok;
  // short response: rows of several heads share a Q tile; a KV group of one tile runs on the single-CTA
  // kernel, several tiles (head dim 256) on the pair kernel, two tiles sharing every key tile
  const bool single = rt.packed && (rt.nq_tiles == 1 || D != 256);
  P.nq_tiles = rt.nq_tiles;
  st = ls::encode_map_rows(&P.a1_map, q, D, R, Hq, rt.bt, rt.bh);
  if (st == LS_OK) st = ls::encode_map_rows(&P.a2_map, d_o, D, R, Hq, rt.bt, rt.bh);
  if (st == LS_OK) st = dense_map(&P.rk_s, k_resp, Hkv, 64, 2);
  if (st == LS_OK) st = dense_map(&P.rv_s, v_resp, Hkv, 64, 2);
  if (st == LS_OK) st = dense_map(&P.rk_m, k_resp, Hkv, 128, 1);
  if (st == LS_OK) st = dense_map(&P.rv_m, v_resp, Hkv, 128, 1);
  if (st == LS_OK) st = ls::pool_map(&P.pk_s, h, 0, 64, 2, false);
  if (st == LS_OK) st = ls::pool_map(&P.pk_s_tail, h, 0, 64, 2, true);
  if (st == LS_OK) st = ls::pool_map(&P.pv_s, h, 1, 64, 2, false);
  if (st == LS_OK) st = ls::pool_map(&P.pv_s_tail, h, 1, 64, 2, true);
  if (st == LS_OK) st = ls::pool_map(&P.pk_m, h, 0, mbox, 1, false);
  if (st == LS_OK) st = ls::pool_map(&P.pk_m_tail, h, 0, mbox, 1, true);
  if (st == LS_OK) st = ls::pool_map(&P.pv_m, h, 1, mbox, 1, false);
  if (st == LS_OK) st = ls::pool_map(&P.pv_m_tail, h, 1, mbox, 1, true);
  if (st != LS_OK) return st;
  if (cudaMemsetAsync(ctl, 0, ctl_bytes, cs) != cudaSuccess) return LS_ERR_CUDA;
  if (single) {
    // short response: one single-CTA work item per (KV head, part, Q tile); K/V pages come from DRAM once
    const int pbox = small_pages ? 64 : 128, pgroups = small_pages ? 1 : 2;
    st = dense_map(&P.b1r_map, k_resp, Hkv, 128, 2);
    if (st == LS_OK) st = dense_map(&P.b2r_map, v_resp, Hkv, 128, 2);
    if (st == LS_OK) st = ls::pool_map(&P.bk_map, h, 0, pbox, pgroups, false);
    if (st == LS_OK) st = ls::pool_map(&P.bk_tail, h, 0, pbox, pgroups, true);
    if (st == LS_OK) st = ls::pool_map(&P.bv_map, h, 1, pbox, pgroups, false);
    if (st == LS_OK) st = ls::pool_map(&P.bv_tail, h, 1, pbox, pgroups, true);
    if (st != LS_OK) return st;
    int64_t grid1 = (int64_t)Hkv * (parts + 1) * rt.nq_tiles;
    P.dq1_ranges = 1;
    if (rt.nq_tiles == 1) {
      P.dq_split = dq_acc + rows * D;      // (see ls_replay_attn_workspace_bytes)
      P.dq1_ranges = ls::dq1_ranges(Hkv, d.prefix_len);
      grid1 = (int64_t)Hkv * P.dq1_ranges;
    }
    st = (D == 128) ? ls::launch_dq1<128>(P, grid1, cs) : ls::launch_dq1<256>(P, grid1, cs);
    if (st == LS_OK && P.dq_split) {
      const int64_t n4 = rows * D / 4;
      ls::dq_reduce_kernel<<<(int)std::min<int64_t>((n4 + 255) / 256, 148 * 16), 256, 0, cs>>>(
          P.dq_split, P.dq1_ranges, n4, prm->scale, static_cast<__nv_bfloat16*>(dq));
      if (cudaGetLastError() != cudaSuccess) st = LS_ERR_CUDA;
    }
  } else {
    const int64_t grid2 = (int64_t)Hkv * (parts + 1) * ((P.nq_tiles + 1) / 2) * 2;
    st = (D == 128) ? ls::launch_dq2<128>(P, grid2, cs) : ls::launch_dq3(P, grid2, cs);
  }
  if (st != LS_OK) return st;

  // ---- dK and dV: rows = keys, columns = queries of the KV group
  st = dense_map(&P.b1r_map, q, Hq, 128, 2);
  if (st == LS_OK) st = dense_map(&P.b2r_map, d_o, Hq, 128, 2);
  if (st != LS_OK) return st;
  const int pg = d.page_size;
  // keys of every suffix block, read through their pages: the sums go into the block's fp32 gradient pages
  for (size_t b = 0; b < h->suffix_blocks.size(); ++b) {
    const ls::SuffixBlock& blk = h->suffix_blocks[b];
    P.keys_paged = 1;
    P.key_page_off = (int)(h->num_logical_pages + blk.first_slot);
    P.key_tokens = blk.tokens;
    P.grad_slot0 = blk.first_slot;
    const int grid_b = Hkv * ((blk.tokens + 127) / 128);
    st = ls::pool_map(&P.a1_map, h, 0, mbox, 1, false);
    if (st == LS_OK) st = ls::pool_map(&P.a2_map, h, 1, mbox, 1, false);
    if (st != LS_OK) return st;
    P.b3r_map = P.b1r_map;
    P.grad = h->dk_grad;
    st = (D == 128) ? ls::launch_kv<128, ls::MODE_DK>(P, grid_b, cs, false)
                    : ls::launch_kv<256, ls::MODE_DK>(P, grid_b, cs, false);
    if (st != LS_OK) return st;
    P.b3r_map = P.b2r_map;
    P.grad = h->dv_grad;
    st = (D == 128) ? ls::launch_kv<128, ls::MODE_DV>(P, grid_b, cs, false)
                    : ls::launch_kv<256, ls::MODE_DV>(P, grid_b, cs, false);
    if (st != LS_OK) return st;
  }
  if (no_resp) return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
  // keys of the response block itself (causal); with LS_FLAG_ADD_SUFFIX_GRAD the gradient pages that later
  // blocks left for this block (its slots start where the suffix now ends) are added
  P.keys_paged = 0;
  P.key_tokens = R;
  P.grad_slot0 = (int)h->suffix_phys.size();
  if (add_grad && P.grad_slot0 + (R + pg - 1) / pg > h->suffix_cap_pages) return LS_ERR_INVALID_ARG;
  const int grid_kv = Hkv * tiles_per_head;
  st = dense_map(&P.a1_map, k_resp, Hkv, 128, 1);
  if (st == LS_OK) st = dense_map(&P.a2_map, v_resp, Hkv, 128, 1);
  if (st != LS_OK) return st;
  P.b3r_map = P.b1r_map;
  P.out = static_cast<__nv_bfloat16*>(dk_resp);
  P.grad = add_grad ? h->dk_grad : nullptr;
  st = (D == 128) ? ls::launch_kv<128, ls::MODE_DK>(P, grid_kv, cs, true) : ls::launch_kv<256, ls::MODE_DK>(P, grid_kv, cs, true);
  if (st != LS_OK) return st;
  P.b3r_map = P.b2r_map;
  P.out = static_cast<__nv_bfloat16*>(dv_resp);
  P.grad = add_grad ? h->dv_grad : nullptr;
  st = (D == 128) ? ls::launch_kv<128, ls::MODE_DV>(P, grid_kv, cs, true) : ls::launch_kv<256, ls::MODE_DV>(P, grid_kv, cs, true);
  if (st != LS_OK) return st;
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

// ---------------------------------------------------------------------------------
// Backward without caller scratch: Delta, the hand-over counters and the running dQ live in a
// fixed array inside the library's device image instead of a caller-provided workspace.
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
  // the handle must belong to the current device: the scratch address is looked up per device
  ls_status_t st = ls::check_handle(h, prm);
  if (st != LS_OK) return st;
  const size_t need = ls_replay_attn_workspace_bytes(h, prm, LS_WORKSPACE_BWD);
  if (need == 0) return LS_ERR_INVALID_ARG;
  if (need > ls::kStaticScratchBytes) return LS_ERR_WORKSPACE;   // shape too large for the built-in scratch
  void* scratch = nullptr;
  st = ls::static_scratch(&scratch);
  if (st != LS_OK) return st;
  // The array keeps the previous call's contents.  The only words that must start at zero are
  // the hand-over counters, which the backward clears itself (a memset node on `stream`, no
  // allocation); Delta and the running dQ are written before they are read.
  return ls_replay_attn_bwd(h, prm, q, k_resp, v_resp, o_f32, lse, d_o, dq, dk_resp, dv_resp, scratch,
                            ls::kStaticScratchBytes, status_dev, stream);
}
