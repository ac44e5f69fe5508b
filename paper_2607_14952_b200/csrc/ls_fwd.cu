// Per-shard replay forward (Eq. qwen-local-attn) for sm_100a.
//
// One CTA owns one work item: (KV head, partial, 128-row Q tile of one query head).
// Partials 0..S-1 are the prefix shards, partial S is the causal response block.
// Work items are ordered KV head -> partial -> Q tile, so CTAs that run together stream
// the same K/V pages and share them through L2.
//
// Warp roles (192 threads):
//   warp 0  producer: walks the shard's page list and issues TMA box loads into a ring
//           of 16 KB chunks, in the exact order the tensor core consumes them
//   warp 1  MMA issuer: S = Q K^T (operands in shared memory) and O += P V (P read from
//           TMEM, V MN-major from shared memory) with tcgen05.mma; owns the TMEM allocation
//   warps 2-5  softmax: one thread per query row (TMEM lane); online softmax with a lazily
//           updated reference maximum, P written back to TMEM as bf16 over the S columns
//
// A CTA owns DVT output channels (all of them for head dims 128 and 256).  The shared-latent
// shape (576/512, V = first 512 channels of the K page) runs as two work items per Q tile,
// one per 256-channel half of O, because O alone would fill all 512 TMEM columns.
//
// TMEM columns: O [0, DVT), S/P buffer 0 [DVT, DVT+128), S/P buffer 1 [DVT+128, DVT+256).
// K chunk  = 128 keys x 64*KSLABS channels (K-major, 128-byte swizzle): k-slices of S.
// V chunk  = VKEYS keys x DVT channels as DVT/64 sub-slabs (MN-major): VKEYS/16 k-steps of PV.
#include "ls_internal.h"
#include "ls_sm100.cuh"

namespace ls {

// How the CTAs of one launch hand their results over (FwdParams::chain_mode):
//   0  every work item writes its own partial (o_r, l_r);
//   1  the `fine` consecutive sub-shards of a shard fold into that shard's partial, in order;
//   2  every part -- the response block first, then the prefix sub-shards, then the suffix
//      blocks -- folds into one composed output (Eq. qwen-global-attn), in that order.
// Folding is the pairwise form of Eq. qwen-lse-parts on normalised values:
//   m = max(l, l_r); a = e^{l-m} + e^{l_r-m}; o = (e^{l-m} o + e^{l_r-m} o_r) / a; l = m + log a.
struct FwdParams {
  CUtensorMap q_map;               // box 64 x 128 tokens x KSLABS channel groups
  CUtensorMap k_map, k_tail_map;   // pool K: box 64 x 128 x KSLABS (pages >= 128 tokens) or 64 x 64 x 1
  CUtensorMap v_map, v_tail_map;   // pool V: box 64 x VKEYS tokens x DVT/64 groups
  CUtensorMap kr_map, vr_map;      // response K (64 x 128 x KSLABS) and V (64 x VKEYS x DVT/64)
  // CTA-pair variant (D = 256): every box is 64 channels x 64 tokens x 2 groups (16 KB)
  CUtensorMap pk2, pk2_tail, pv2, pv2_tail, rk2, rv2;
  // the odd ninth channel group of the 576-wide key: 64 channels x 64 tokens x 1 group (8 KB)
  CUtensorMap pk1, pk1_tail, rk1;
  const int32_t* part_pages;
  const int32_t* part_page_offset;
  const int32_t* part_tail_slot;
  const int64_t* part_tokens;
  float* o_out;        // modes 0, 1: prefix partials [S_out, R, Hq, dv]; mode 2: the running output [R, Hq, dv]
  float* lse_out;
  float* o_resp;       // modes 0, 1: the response block's partial [R, Hq, dv]
  float* lse_resp;
  __nv_bfloat16* o_bf16;   // mode 2: composed output in bf16, written by the last link (nullable)
  float* lse_aux;      // two O tiles per Q tile: running l of the second tile's chain
  int* ctl;            // hand-over control words (ticket, abort, counters) or NULL
  int32_t* status;
  long long* timing;   // diagnostic builds only
  int R, Hq, Hkv, g, parts, pg_shift, nq_tiles, num_phys_pages;
  // Q tiles of a KV group (RowTiling): tile q covers bt tokens from (q % tiles_tok) * bt of bh heads from
  // (q / tiles_tok) * bh; its row r is head r / bt, token r % bt.  Long responses: bt = 128, bh = 1.
  int bt, bh, tiles_tok;
  int chain_mode, fine;
  int no_resp;    // 1: the response block is left out (its partial is written as empty)
  int dv_total;   // channels of one output row (DVT times the number of O tiles)
  int q_bytes;    // bytes the Q loads deliver
  int ablate;     // diagnostic builds only (LS_DBG_ABLATE_*)
  float scale, scale_log2;
};

// Build with -DLS_TIMING to make CTA 0 write per-role cycle counts (time spent in each kind
// of wait, and in total) into the buffer given to ls_debug_timing_buffer; a profiling aid.
#ifdef LS_TIMING
#define LS_TWAIT(acc, expr) ([&] { const long long t0_ = clock64(); const bool r_ = (expr); (acc) += clock64() - t0_; return r_; }())
#define LS_TDUMP(slot, val) do { if (blockIdx.x == 0 && p.timing) p.timing[(slot)] = (val); } while (0)
#define LS_ABLATE(bit) ((p.ablate & (bit)) != 0)
#else
#define LS_TWAIT(acc, expr) (expr)
#define LS_TDUMP(slot, val) do { } while (0)
#define LS_ABLATE(bit) false
#endif

// One work item: which keys (part), which Q rows, and where the result goes.
struct FwdItem {
  int kvh, part, qunit, link;
  bool is_resp, chained, first, last;
};
__device__ __forceinline__ FwdItem fwd_item(const FwdParams& p, int idx, int n_qunits) {
  FwdItem it;
  it.qunit = idx % n_qunits;
  idx /= n_qunits;
  const int slots = p.parts + 1;
  const int slot = idx % slots;
  it.kvh = idx / slots;
  if (p.chain_mode == 2) {
    it.link = slot;
    it.is_resp = slot == 0;
    it.part = it.is_resp ? p.parts : slot - 1;
    it.chained = true;
    it.first = slot == 0;
    it.last = slot == p.parts;
  } else {
    it.is_resp = slot == p.parts;
    it.part = slot;
    it.chained = p.chain_mode == 1 && !it.is_resp;
    it.link = it.chained ? slot % p.fine : 0;
    it.first = it.link == 0;
    it.last = false;
  }
  return it;
}
// index of the partial that receives the item's rows, and of its hand-over counter
__device__ __forceinline__ int fwd_out_part(const FwdParams& p, const FwdItem& it) {
  return (p.chain_mode == 2 || it.is_resp) ? 0 : (p.chain_mode == 1 ? it.part / p.fine : it.part);
}
__device__ __forceinline__ int fwd_chain_index(const FwdParams& p, const FwdItem& it, int qtile) {
  const int group = p.chain_mode == 2 ? it.kvh : it.kvh * (p.parts / p.fine) + it.part / p.fine;
  return group * p.nq_tiles + qtile;
}

// One row thread's share of the epilogue: its (unnormalised) accumulator row in TMEM, the
// row's running sum l and scaled reference maximum, normalised and either stored (fold =
// false) or folded into the value already there.  Rows whose own partial weighs nothing
// leave the running value untouched.
template <int DV>
__device__ __forceinline__ void fwd_store_row(uint32_t tmem_row, bool have_acc, float l, float m_scaled, bool fold,
                                              float* o_dst, float* lse_dst, bool write_lse, __nv_bfloat16* bf_dst,
                                              bool row_ok, bool chained, bool chain_last) {
  const bool own = have_acc && l > 0.f;
  const float lse_own = own ? m_scaled + logf(l) : -INFINITY;
  float c_own = own ? 1.0f / l : 0.f, c_run = 0.f, lse_new = lse_own;
  if (fold) {
    const float lse_run = row_ok ? __ldcg(lse_dst) : -INFINITY;
    const float m = fmaxf(lse_run, lse_own);
    if (m == -INFINITY) {
      c_own = 0.f;
    } else {
      const float w_run = expf(lse_run - m), w_own = expf(lse_own - m);
      const float inv_a = 1.0f / (w_run + w_own);
      c_run = w_run * inv_a;
      c_own *= w_own * inv_a;
      lse_new = m + logf(w_run + w_own);
    }
  }
  const bool store = row_ok && (!fold || c_own != 0.f || bf_dst != nullptr);
  const bool load_run = fold && c_run != 0.f;
  // the running value of a chain is kept in L2 past the K/V stream; the last link hands it back
  const uint64_t pol = (chain_last || !chained) ? l2_policy_evict_first() : l2_policy_evict_last();
#pragma unroll 1
  for (int c = 0; c < DV; c += 32) {
    uint32_t o[32];
    if (have_acc) {
      tmem_ld32(tmem_row + c, o);
      tc_wait_ld32(o);
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) o[j] = 0u;
    }
    if (store) {
      float4 run[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        run[j] = load_run ? ld_cg_hint(reinterpret_cast<const float4*>(o_dst + c) + j, pol) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float4 v;
        v.x = fmaf(c_run, run[j].x, c_own * __uint_as_float(o[4 * j]));
        v.y = fmaf(c_run, run[j].y, c_own * __uint_as_float(o[4 * j + 1]));
        v.z = fmaf(c_run, run[j].z, c_own * __uint_as_float(o[4 * j + 2]));
        v.w = fmaf(c_run, run[j].w, c_own * __uint_as_float(o[4 * j + 3]));
        if (chained) st_hint(reinterpret_cast<float4*>(o_dst + c) + j, v, pol);
        else *(reinterpret_cast<float4*>(o_dst + c) + j) = v;
        if (bf_dst) {
          uint2 pk;
          pk.x = pack_bf16(v.x, v.y);
          pk.y = pack_bf16(v.z, v.w);
          *(reinterpret_cast<uint2*>(bf_dst + c) + j) = pk;
        }
      }
    }
  }
  if (store && write_lse) *lse_dst = lse_new;
}

constexpr int kFwdThreads = 192;
constexpr float kRescaleLog2 = 8.0f;   // the reference max lags the true max by at most 2^8

template <int DK, int DVT>
struct FwdCfg {
  static constexpr int CHUNK = (DK == 256) ? 32768 : 16384;   // bytes per ring slot
  static constexpr int KSLABS = CHUNK / 16384;     // 64-channel slabs (128 keys x 128 B) per K chunk
  static constexpr int KCH = (DK / 64) / KSLABS;   // K chunks per 128-key tile
  static constexpr int VKEYS = CHUNK / (DVT * 2);  // keys per V chunk
  static constexpr int NVCH = 128 / VKEYS;         // V chunks per tile
  static constexpr int VSUB = DVT / 64;            // sub-slabs (VKEYS rows x 128 B) per V chunk
  static_assert(VSUB * VKEYS * 128 == CHUNK && VKEYS % 16 == 0 && VKEYS <= 64, "a V chunk fills one ring slot");
  static constexpr int RING = (DK == 256) ? 4 : (DK == 128) ? 10 : 5;
  static constexpr int Q_BYTES = (DK / 64) * 16384;
  static constexpr int SMEM_BYTES = 1024 + Q_BYTES + RING * CHUNK + 512;
};

// Row-thread wait: the warp leaves together (the TMEM loads and votes that follow need every lane).
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
}

template <int DK, int DVT, int NDV>
__global__ void __launch_bounds__(kFwdThreads, 1) fwd_kernel(const __grid_constant__ FwdParams p) {
  using C = FwdCfg<DK, DVT>;
  constexpr int DV = DVT;   // O columns held by this CTA
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_smem = smem;
  uint8_t* ring = smem + C::Q_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + C::RING * C::CHUNK);
  uint64_t* q_full = bars;
  uint64_t* full = bars + 1;
  uint64_t* empty = full + C::RING;
  uint64_t* s_full = empty + C::RING;   // [2]
  uint64_t* p_full = s_full + 2;        // [2]
  uint64_t* pv_done = p_full + 2;       // one phase per tile: O += P V of that tile finished
  uint64_t* o_final = pv_done + 1;      // the last tile's P V finished
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(o_final + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  int* work_idx = const_cast<int*>(abort_flag) + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  long long tw0 = 0, tw1 = 0, tw2 = 0;   // wait-time accumulators (only used with LS_TIMING)
  (void)tw0; (void)tw1; (void)tw2;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int i = 0; i < C::RING; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    mbar_init(&s_full[0], 1);
    mbar_init(&s_full[1], 1);
    mbar_init(&p_full[0], 128);
    mbar_init(&p_full[1], 128);
    mbar_init(pv_done, 1);
    mbar_init(o_final, 1);
    *abort_flag = 0;
    // work items are handed out in launch order of the CTAs that ask, so an item never waits
    // for one that no CTA has started
    *work_idx = p.ctl ? atomicAdd(p.ctl, 1) : (int)blockIdx.x;
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
  const uint32_t tmem_o = tmem_base;
  const uint32_t tmem_s0 = tmem_base + DV;

  // ---- work item
  int idx = *work_idx;
  const int dvh = idx % NDV;            // which DVT-wide slice of the value channels
  idx /= NDV;
  const FwdItem it = fwd_item(p, idx, p.nq_tiles);
  const int qtile = it.qunit, part = it.part, kvh = it.kvh;
  const int h = kvh * p.g + (qtile / p.tiles_tok) * p.bh;      // first head and token of the tile
  const int t0 = (qtile % p.tiles_tok) * p.bt;
  const bool is_resp = it.is_resp;
  int64_t tokens;
  int page_off = 0, n_pages = 0, tail_slot = -1;
  if (is_resp) {
    tokens = p.no_resp ? 0 : min(p.R, t0 + p.bt);      // keys 0 .. last row of this tile (none when the block is left out)
  } else {
    tokens = p.part_tokens[part];
    page_off = p.part_page_offset[part];
    n_pages = p.part_page_offset[part + 1] - page_off;
    tail_slot = p.part_tail_slot[part];
  }
  const int n_tiles = (int)((tokens + 127) / 128);

  if (warp == 0) {
    // =========================================================== producer (one thread)
    if (lane == 0 && n_tiles > 0) {
      const bool no_loads = LS_ABLATE(LS_DBG_ABLATE_LOADS);
      mbar_arrive_expect_tx(q_full, p.q_bytes);
      for (int c = 0; c < DK / 64; ++c) tma_load_5d(q_smem + c * 16384, &p.q_map, q_full, 0, t0, c, h, 0);

      const int32_t* pages = p.part_pages + page_off;
      const int pg_mask = (1 << p.pg_shift) - 1;
      const bool small_pages = p.pg_shift == 6;          // 64-token pages: a tile spans two pages
      // physical page of the part's page slot; past the part's last page the coordinate points
      // beyond the pool and TMA fills zeros
      auto fetch = [&](int slot_idx) -> int {
        return (slot_idx < n_pages) ? __ldg(pages + slot_idx) : p.num_phys_pages;
      };
      uint32_t slot = 0, phase = 0, issued = 0;
      bool ok = true;
      auto acquire = [&]() -> uint8_t* {
        ok = ok && LS_TWAIT(tw0, mbar_wait(&empty[slot], phase ^ 1, abort_flag));
        uint8_t* dst = ring + slot * C::CHUNK;
        if (ok) {
          if (no_loads) mbar_arrive(&full[slot]);
          else mbar_arrive_expect_tx(&full[slot], C::CHUNK);
        }
        return dst;
      };
      auto advance = [&]() {
        ++issued;
        if (++slot == (uint32_t)C::RING) { slot = 0; phase ^= 1; }
      };
      // K of one tile: KCH chunks of 128 keys x (64 * KSLABS) channels
      auto load_k = [&](int tile, int pa, int pb) {
        const int tok = tile * 128;
        for (int c = 0; c < C::KCH; ++c) {
          uint8_t* dst = acquire();
          if (ok && !no_loads) {
            if (is_resp) {
              tma_load_5d(dst, &p.kr_map, &full[slot], 0, tok, c * C::KSLABS, kvh, 0);
            } else if (!small_pages) {
              const CUtensorMap* m = ((tok >> p.pg_shift) == tail_slot) ? &p.k_tail_map : &p.k_map;
              tma_load_5d(dst, m, &full[slot], 0, tok & pg_mask, c * C::KSLABS, kvh, pa);
            } else {
              const int sa = tok >> 6;
              const CUtensorMap* ma = (sa == tail_slot) ? &p.k_tail_map : &p.k_map;
              const CUtensorMap* mb = (sa + 1 == tail_slot) ? &p.k_tail_map : &p.k_map;
              for (int s = 0; s < C::KSLABS; ++s) {
                tma_load_5d(dst + s * 16384, ma, &full[slot], 0, 0, c * C::KSLABS + s, kvh, pa);
                tma_load_5d(dst + s * 16384 + 8192, mb, &full[slot], 0, 0, c * C::KSLABS + s, kvh, pb);
              }
            }
          }
          advance();
        }
      };
      // V of one tile: NVCH chunks of VKEYS keys x DVT channels (channel groups dvh*VSUB ..)
      auto load_v = [&](int tile, int pa, int pb) {
        for (int r = 0; r < C::NVCH; ++r) {
          uint8_t* dst = acquire();
          if (ok && !no_loads) {
            const int tok = tile * 128 + r * C::VKEYS;
            if (is_resp) {
              tma_load_5d(dst, &p.vr_map, &full[slot], 0, tok, dvh * C::VSUB, kvh, 0);
            } else {
              const CUtensorMap* m = ((tok >> p.pg_shift) == tail_slot) ? &p.v_tail_map : &p.v_map;
              tma_load_5d(dst, m, &full[slot], 0, tok & pg_mask, dvh * C::VSUB, kvh,
                          (small_pages && r * C::VKEYS >= 64) ? pb : pa);
            }
          }
          advance();
        }
      };
      const long long t_begin_p = clock64();
      (void)t_begin_p;
      // page ids of tile i: slots (128 i) >> pg_shift and, for 64-token pages, the next one
      int pa0 = 0, pb0 = 0, pa1 = 0, pb1 = 0;
      if (!is_resp) {
        pa0 = fetch(0);
        pb0 = small_pages ? fetch(1) : pa0;
        if (n_tiles > 1) {
          pa1 = fetch(128 >> p.pg_shift);
          pb1 = small_pages ? fetch(3) : pa1;
        }
      }
      load_k(0, pa0, pb0);
      for (int i = 0; i < n_tiles; ++i) {
        int pa2 = 0, pb2 = 0;                       // prefetched two tiles ahead, used next iteration
        if (!is_resp && i + 2 < n_tiles) {
          const int s2 = ((i + 2) * 128) >> p.pg_shift;
          pa2 = fetch(s2);
          pb2 = small_pages ? fetch(s2 + 1) : pa2;
        }
        if (i + 1 < n_tiles) load_k(i + 1, pa1, pb1);
        load_v(i, pa0, pb0);
        pa0 = pa1; pb0 = pb1; pa1 = pa2; pb1 = pb2;
      }
      LS_TDUMP(0, tw0);
      LS_TDUMP(1, clock64() - t_begin_p);
      // On an aborted run, wait (bounded) until every copy this thread started has landed.
      if (*abort_flag) {
        for (uint32_t s = 0; s < (uint32_t)C::RING && s < issued; ++s) {
          const uint32_t last = ((issued - 1 - s) / C::RING) * C::RING + s;   // last chunk index in slot s
          const uint64_t t_start = globaltimer_ns();
          while (!mbar_try_wait(&full[s], (last / C::RING) & 1, 1000) && globaltimer_ns() - t_start < 100000000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // =========================================================== MMA issuer (one thread)
    if (lane == 0 && n_tiles > 0) {
      constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);
      constexpr uint32_t idesc_pv = make_idesc(128, DV, 0, 1);
      constexpr uint32_t hi = sdesc_hi(1024);
      const uint32_t q_lo = sdesc_lo(smem_u32(q_smem), 16);
      const uint32_t ring_k_lo = sdesc_lo(smem_u32(ring), 16);       // K-major chunk
      const uint32_t ring_v_lo = sdesc_lo(smem_u32(ring), C::VKEYS * 128);   // MN-major chunk: sub-slab pitch
      uint32_t slot = 0, phase = 0;
      const bool no_mma = LS_ABLATE(LS_DBG_ABLATE_MMA);
      bool ok = mbar_wait(q_full, 0, abort_flag);
      const long long t_begin = clock64();
      (void)t_begin;
      auto advance = [&]() {
        if (++slot == (uint32_t)C::RING) { slot = 0; phase ^= 1; }
      };
      auto issue_s = [&](int tile) {
        const uint32_t d = tmem_s0 + (tile & 1) * 128;
#pragma unroll
        for (int c = 0; c < C::KCH; ++c) {
          ok = ok && LS_TWAIT(tw0, mbar_wait(&full[slot], phase, abort_flag));
          if (!ok) return;
          tc_fence_after();
          const uint32_t b_lo = ring_k_lo + slot * (C::CHUNK >> 4);
          if (!no_mma) {
#pragma unroll
            for (int s = 0; s < C::KSLABS; ++s)
#pragma unroll
              for (int k = 0; k < 4; ++k)
                mma_ss(d, sdesc(q_lo + (((c * C::KSLABS + s) * 16384 + k * 32) >> 4), hi),
                       sdesc(b_lo + ((s * 16384 + k * 32) >> 4), hi), idesc_s, (c | s | k) != 0);
          }
          mma_commit(&empty[slot]);
          advance();
        }
        mma_commit(&s_full[tile & 1]);
      };
      auto issue_pv = [&](int tile) {
        const uint32_t a_base = tmem_s0 + (tile & 1) * 128;   // P over the S columns
#pragma unroll
        for (int r = 0; r < C::NVCH; ++r) {
          ok = ok && LS_TWAIT(tw1, mbar_wait(&full[slot], phase, abort_flag));
          if (!ok) return;
          tc_fence_after();
          const uint32_t b_lo = ring_v_lo + slot * (C::CHUNK >> 4);
          if (!no_mma) {
#pragma unroll
            for (int kk = 0; kk < C::VKEYS / 16; ++kk)
              mma_ts(tmem_o, a_base + (r * (C::VKEYS / 16) + kk) * 8, sdesc(b_lo + ((kk * 2048) >> 4), hi),
                     idesc_pv, (tile | r | kk) != 0);
          }
          mma_commit(&empty[slot]);
          advance();
        }
        mma_commit(pv_done);
        if (tile == n_tiles - 1) mma_commit(o_final);
      };
      if (ok) issue_s(0);
      for (int i = 0; i < n_tiles && ok; ++i) {
        if (i + 1 < n_tiles) issue_s(i + 1);
        ok = ok && LS_TWAIT(tw2, mbar_wait(&p_full[i & 1], (i >> 1) & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        issue_pv(i);
      }
      LS_TDUMP(8, tw0);
      LS_TDUMP(9, tw1);
      LS_TDUMP(10, tw2);
      LS_TDUMP(11, clock64() - t_begin);
    }
  } else {
    // =========================================================== softmax + epilogue
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    // this thread's (token, head) inside the tile of bt tokens x bh heads
    const int hj = row / p.bt;
    const int t = t0 + row - hj * p.bt;
    const bool row_ok = hj < p.bh && t < p.R && h + hj < (kvh + 1) * p.g;
    const int hr = min(h + hj, p.Hq - 1);
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    const size_t out_row = ((size_t)fwd_out_part(p, it) * p.R + (size_t)min(t, p.R - 1)) * p.Hq + hr;
    const bool to_resp = is_resp && p.chain_mode != 2;
    float* o_dst = (to_resp ? p.o_resp : p.o_out) + out_row * p.dv_total + dvh * DVT;
    float* lse_dst = (to_resp ? p.lse_resp : p.lse_out) + out_row;
    if (dvh != 0 && it.chained) lse_dst = p.lse_aux + out_row;     // the second O tile's chain keeps its own copy of l
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    if (n_tiles > 0) {
      // last visible key index of this row inside this partial
      const int64_t lim = is_resp ? (int64_t)min(t, p.R - 1) : tokens - 1;
      const long long t_begin_sm = clock64();
      (void)t_begin_sm;
      const float thresh = kRescaleLog2 / p.scale_log2;
      for (int i = 0; i < n_tiles && ok; ++i) {
        const uint32_t ts = tmem_s0 + (i & 1) * 128 + lane_sel;
        ok = LS_TWAIT(tw0, mbar_wait_warp(&s_full[i & 1], (i >> 1) & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        if (LS_ABLATE(LS_DBG_ABLATE_SOFTMAX)) {
          tc_fence_before();
          mbar_arrive(&p_full[i & 1]);
          continue;
        }
        uint32_t sr[128];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(ts + c * 32, sr + c * 32);
#pragma unroll
        for (int c = 0; c < 4; ++c) tc_wait_ld32(sr + c * 32);
        float* s = reinterpret_cast<float*>(sr);
        const int key0 = i * 128;
        if (__any_sync(0xffffffffu, (int64_t)key0 + 127 > lim)) {
#pragma unroll
          for (int j = 0; j < 128; ++j)
            if ((int64_t)key0 + j > lim) s[j] = -INFINITY;
        }
        float mx0 = s[0], mx1 = s[1], mx2 = s[2], mx3 = s[3];
#pragma unroll
        for (int j = 4; j < 128; j += 4) {
          mx0 = fmaxf(mx0, s[j]);
          mx1 = fmaxf(mx1, s[j + 1]);
          mx2 = fmaxf(mx2, s[j + 2]);
          mx3 = fmaxf(mx3, s[j + 3]);
        }
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        if (i == 0) {
          m_ref = (mx == -INFINITY) ? 0.f : mx;
        } else if (__any_sync(0xffffffffu, row_ok && mx > m_ref + thresh)) {   // (rows outside the tile hold stale bytes: they must not steer the warp)
          // rare: raise the reference maximum and rescale the running sum and O
          ok = LS_TWAIT(tw1, mbar_wait_warp(pv_done, (i - 1) & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
          const float m_new = fmaxf(m_ref, mx);
          const float f = ex2((m_ref - m_new) * p.scale_log2);
          m_ref = m_new;
          l *= f;
#pragma unroll 1
          for (int c = 0; c < DV; c += 32) {
            uint32_t o[32];
            tmem_ld32(tmem_o + lane_sel + c, o);
            tc_wait_ld32(o);
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * f);
            tmem_st32(tmem_o + lane_sel + c, o);
          }
          tc_wait_st();
        }
        const float neg_m = -m_ref * p.scale_log2;
        uint32_t pk[64];
        float l0 = 0.f, l1 = 0.f;
#pragma unroll
        for (int j = 0; j < 128; j += 2) {
          const float p0 = ex2(fmaf(s[j], p.scale_log2, neg_m));
          const float p1 = ex2(fmaf(s[j + 1], p.scale_log2, neg_m));
          l0 += p0;
          l1 += p1;
          pk[j >> 1] = pack_bf16(p0, p1);
        }
        l += l0 + l1;
        tmem_st32(ts, pk);
        tmem_st32(ts + 32, pk + 32);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(&p_full[i & 1]);
      }
      // (pv_done may still be two phases behind here, where a parity wait would alias)
      if (threadIdx.x == 64) {
        LS_TDUMP(16, tw0);
        LS_TDUMP(17, tw1);
        LS_TDUMP(18, clock64() - t_begin_sm);
      }
      if (ok) ok = mbar_wait_warp(o_final, 0, abort_flag);
      if (ok) tc_fence_after();
    }
    // ---- epilogue: store this partial, or fold it into the running value of its chain
    int* counter = it.chained ? p.ctl + kChainHeaderInts + fwd_chain_index(p, it, qtile) * NDV + dvh : nullptr;
    const bool fold = it.chained && !it.first;
    if (ok && fold) ok = __all_sync(0xffffffffu, chain_wait(counter, it.link, p.ctl, abort_flag));
    if (ok)
      fwd_store_row<DV>(tmem_o + lane_sel, n_tiles > 0, l, m_ref * p.scale, fold, o_dst, lse_dst,
                        dvh == 0 || it.chained, (it.last && p.o_bf16) ? p.o_bf16 + out_row * p.dv_total + dvh * DVT : nullptr,
                        row_ok, it.chained, it.chained && (p.chain_mode == 2 ? it.last : it.link == p.fine - 1));
    if (it.chained) {
      const bool all_ok = bar_and(2, 128, ok);     // every row of the tile is written
      if (row == 0 && all_ok) chain_publish(counter, it.link + 1);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
  if (threadIdx.x == 0 && *abort_flag) {
    if (p.status) atomicExch(p.status, (int)LS_ERR_TIMEOUT);
    if (p.ctl) st_relaxed_gpu(p.ctl + 1, 1);    // ends every other chain wait of this launch
  }
}

// ---------------------------------------------------------------------------------
// Forward on CTA pairs (cta_group::2), head dim 256 and the 576/512 shape.  Two neighbouring SMs
// take two Q tiles of the same (KV head, partial) and stream the keys once between them: for S
// each CTA loads 64 of the 128 keys of a tile, for P V each loads 128 of the 256 value channels,
// so shared-memory writes and L2 reads halve and the ring covers more tiles.  One thread of the
// even CTA issues all MMAs (256 rows); completions are multicast to both CTAs' barriers; the odd
// CTA's softmax warps report P to the even CTA's barrier.  Chunks are 16 KB: 64 tokens x 128
// channels (the ninth 64-channel group of a 576-wide key travels alone, 8 KB in a slot of its own).
// With 512 value channels a pair of Q tiles is NDV = 2 work items, one per 256-channel half of O
// (O of 128 rows x 512 channels alone would fill the 512 TMEM columns).
// ---------------------------------------------------------------------------------
template <int DK>
struct Fwd2Cfg {
  static constexpr int KG = DK / 64;                  // 64-channel groups of a key
  static constexpr int NKC = (KG + 1) / 2;            // key chunks per tile and CTA
  static constexpr int CHUNK = 16384;
  static constexpr int RING = DK == 256 ? 8 : 5;
  static constexpr int Q_BYTES = KG * 16384;
  static constexpr int SMEM_BYTES = 1024 + Q_BYTES + RING * CHUNK + 512;
};

template <int DK, int NDV>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kFwdThreads, 1)
    fwd2_kernel(const __grid_constant__ FwdParams p) {
  using C = Fwd2Cfg<DK>;
  constexpr int DV = 256;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_smem = smem;
  uint8_t* ring = smem + C::Q_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + C::RING * C::CHUNK);
  uint64_t* q_full = bars;              // (even CTA) both CTAs' Q tiles landed
  uint64_t* full = bars + 1;            // (even CTA) both halves of a chunk landed
  uint64_t* empty = full + C::RING;     // (each CTA)
  uint64_t* s_full = empty + C::RING;   // [2] (each CTA)
  uint64_t* p_full = s_full + 2;        // [2] (even CTA) P of both CTAs in TMEM: 8 warp arrivals
  uint64_t* pv_done = p_full + 2;       // (each CTA) one phase per tile
  uint64_t* o_final = pv_done + 1;      // (each CTA)
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(o_final + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  int* work_idx = const_cast<int*>(abort_flag) + 1;   // (even CTA) the pair's work item

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  long long tw0 = 0, tw1 = 0, tw2 = 0;   // wait-time accumulators (only used with LS_TIMING)
  const long long t_begin = clock64();
  (void)tw0; (void)tw1; (void)tw2; (void)t_begin;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int i = 0; i < C::RING; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    mbar_init(&s_full[0], 1);
    mbar_init(&s_full[1], 1);
    mbar_init(&p_full[0], 8);
    mbar_init(&p_full[1], 8);
    mbar_init(pv_done, 1);
    mbar_init(o_final, 1);
    *abort_flag = 0;
    // work items are handed out in launch order of the pairs that ask (see chain_wait)
    if (leader) *work_idx = p.ctl ? atomicAdd(p.ctl, 1) : (int)(blockIdx.x >> 1);
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
  const uint32_t tmem_o = tmem_base;
  const uint32_t tmem_s0 = tmem_base + DV;

  // ---- work item of the pair, and this CTA's Q tile
  const int npairs = (p.nq_tiles + 1) / 2;
  int widx = (int)ld_shared_cluster_u32(mapa_u32(smem_u32(work_idx), 0));
  const int dvh = widx % NDV;           // which 256-wide slice of the value channels
  widx /= NDV;
  const FwdItem it = fwd_item(p, widx, npairs);
  const int pairi = it.qunit, part = it.part, kvh = it.kvh;
  const bool is_resp = it.is_resp;
  auto tile_of = [&](int qt, int& hh, int& r0) {
    if (qt < p.nq_tiles) {
      hh = kvh * p.g + (qt / p.tiles_tok) * p.bh;     // tile of bt tokens x bh heads (RowTiling)
      r0 = (qt % p.tiles_tok) * p.bt;
    } else {                                 // odd tile count: the pair's second CTA works on zero rows
      hh = kvh * p.g + p.g - 1;
      r0 = p.tiles_tok * p.bt;               // token coordinate past R: TMA delivers zeros
    }
  };
  const int qtile = 2 * pairi + (int)rank;
  int h, t0, h_o, t0_o;
  tile_of(qtile, h, t0);
  tile_of(2 * pairi + 1 - (int)rank, h_o, t0_o);
  int64_t tokens;
  int page_off = 0, n_pages = 0, tail_slot = -1;
  if (is_resp) {
    tokens = p.no_resp ? 0 : min(p.R, max(t0, t0_o) + p.bt);  // both CTAs walk the longer causal range
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
      if (leader) mbar_arrive_expect_tx(q_full, 2 * p.q_bytes);
      for (int c = 0; c < C::KG; ++c) tma_load_5d_pair(q_smem + c * 16384, &p.q_map, q_full, 0, t0, c, h, 0);
      const int32_t* pages = p.part_pages + page_off;
      const int pg_mask = (1 << p.pg_shift) - 1;
      auto page_at = [&](int tok) -> int {
        if (is_resp) return 0;
        const int ps = tok >> p.pg_shift;
        return (ps < n_pages) ? __ldg(pages + ps) : p.num_phys_pages;   // past the end: TMA fills zeros
      };
      uint32_t slot = 0, phase = 0, issued = 0;
      bool ok = true;
      // one chunk: 64 tokens starting at `tok` x channel groups [grp, grp + 2) of K (which = 0) or V;
      // single: the lone last group of an odd group count (8 KB)
      auto load = [&](int which, int tok, int grp, int page, bool single) {
        ok = ok && LS_TWAIT(tw0, mbar_wait(&empty[slot], phase ^ 1, abort_flag));
        if (ok) {
          if (leader) mbar_arrive_expect_tx(&full[slot], single ? C::CHUNK : 2 * C::CHUNK);
          uint8_t* dst = ring + slot * C::CHUNK;
          if (is_resp) {
            tma_load_5d_pair(dst, which ? &p.rv2 : (single ? &p.rk1 : &p.rk2), &full[slot], 0, tok, grp, kvh, 0);
          } else {
            const bool tail = (tok >> p.pg_shift) == tail_slot;
            const CUtensorMap* m = which    ? (tail ? &p.pv2_tail : &p.pv2)
                                   : single ? (tail ? &p.pk1_tail : &p.pk1)
                                            : (tail ? &p.pk2_tail : &p.pk2);
            tma_load_5d_pair(dst, m, &full[slot], 0, tok & pg_mask, grp, kvh, page);
          }
        }
        ++issued;
        if (++slot == (uint32_t)C::RING) { slot = 0; phase ^= 1; }
      };
      // K of tile i for S: this CTA's 64 keys, chunks of 128 channels.
      // V of tile i for P V: both 64-key halves, this CTA's 128 of the work item's 256 channels.
      auto load_k = [&](int i, int pa, int pb) {
        const int tok = i * 128 + (int)rank * 64;
        const int pg = rank ? pb : pa;
#pragma unroll
        for (int c = 0; c < C::NKC; ++c) load(0, tok, 2 * c, pg, 2 * c + 1 == C::KG);
      };
      auto load_v = [&](int i, int pa, int pb) {
        load(1, i * 128, 4 * dvh + 2 * (int)rank, pa, false);
        load(1, i * 128 + 64, 4 * dvh + 2 * (int)rank, pb, false);
      };
      // pages of the two 64-key halves of tile i (equal unless the pages hold 64 tokens)
      int pa0 = page_at(0), pb0 = page_at(64), pa1 = page_at(128), pb1 = page_at(192);
      load_k(0, pa0, pb0);
      for (int i = 0; i < n_tiles; ++i) {
        const int pa2 = (i + 2 < n_tiles) ? page_at((i + 2) * 128) : 0;        // used next round
        const int pb2 = (i + 2 < n_tiles) ? page_at((i + 2) * 128 + 64) : 0;
        if (i + 1 < n_tiles) load_k(i + 1, pa1, pb1);
        load_v(i, pa0, pb0);
        pa0 = pa1; pb0 = pb1; pa1 = pa2; pb1 = pb2;
      }
      LS_TDUMP(0, tw0);
      LS_TDUMP(1, clock64() - t_begin);
      if (*abort_flag && leader) {   // aborted: wait (bounded) for the copies credited to this CTA's barriers
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
      constexpr uint32_t idesc_s = make_idesc(256, 128, 0, 0);
      constexpr uint32_t idesc_pv = make_idesc(256, 256, 0, 1);
      constexpr uint32_t hi = sdesc_hi(1024);
      const uint32_t q_lo = sdesc_lo(smem_u32(q_smem), 16);
      const uint32_t ring_k_lo = sdesc_lo(smem_u32(ring), 16);       // K-major: 2 slabs of 64 keys x 64 channels
      const uint32_t ring_v_lo = sdesc_lo(smem_u32(ring), 8192);     // MN-major: 2 groups of 64 channels x 64 keys
      uint32_t slot = 0, phase = 0;
      bool ok = mbar_wait(q_full, 0, abort_flag);
      auto advance = [&]() {
        if (++slot == (uint32_t)C::RING) { slot = 0; phase ^= 1; }
      };
      auto issue_s = [&](int tile) {
        const uint32_t d = tmem_s0 + (tile & 1) * 128;
#pragma unroll
        for (int c = 0; c < C::NKC; ++c) {
          ok = ok && LS_TWAIT(tw1, mbar_wait(&full[slot], phase, abort_flag));
          if (!ok) return;
          tc_fence_after();
          const uint32_t b_lo = ring_k_lo + slot * (C::CHUNK >> 4);
#pragma unroll
          for (int s2 = 0; s2 < 2; ++s2) {
            if (2 * c + s2 >= C::KG) break;
#pragma unroll
            for (int k = 0; k < 4; ++k)
              mma_ss_pair(d, sdesc(q_lo + (((2 * c + s2) * 16384 + k * 32) >> 4), hi),
                          sdesc(b_lo + ((s2 * 8192 + k * 32) >> 4), hi), idesc_s, (c | s2 | k) != 0);
          }
          mma_commit_pair(&empty[slot]);
          advance();
        }
        mma_commit_pair(&s_full[tile & 1]);
      };
      auto issue_pv = [&](int tile) {
        const uint32_t a_base = tmem_s0 + (tile & 1) * 128;   // P over the S columns
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          ok = ok && LS_TWAIT(tw1, mbar_wait(&full[slot], phase, abort_flag));
          if (!ok) return;
          tc_fence_after();
          const uint32_t b_lo = ring_v_lo + slot * (C::CHUNK >> 4);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            mma_ts_pair(tmem_o, a_base + (r * 4 + kk) * 8, sdesc(b_lo + ((kk * 2048) >> 4), hi), idesc_pv,
                        (tile | r | kk) != 0);
          mma_commit_pair(&empty[slot]);
          advance();
        }
        mma_commit_pair(pv_done);
        if (tile == n_tiles - 1) mma_commit_pair(o_final);
      };
      if (ok) issue_s(0);
      for (int i = 0; i < n_tiles && ok; ++i) {
        if (i + 1 < n_tiles) issue_s(i + 1);
        ok = ok && LS_TWAIT(tw2, mbar_wait(&p_full[i & 1], (i >> 1) & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        issue_pv(i);
      }
      LS_TDUMP(9, tw1);
      LS_TDUMP(10, tw2);
      LS_TDUMP(11, clock64() - t_begin);
      LS_TDUMP(12, n_tiles);
    }
  } else {
    // =========================================================== softmax + epilogue (both CTAs)
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int hj = row / p.bt;               // this thread's (token, head) inside the tile of bt tokens x bh heads
    const int t = t0 + row - hj * p.bt;
    const int hr = min(h + hj, p.Hq - 1);
    const bool tile_ok = qtile < p.nq_tiles;
    const bool row_ok = tile_ok && hj < p.bh && t < p.R && h + hj < (kvh + 1) * p.g;
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    const size_t out_row = ((size_t)fwd_out_part(p, it) * p.R + (size_t)min(t, p.R - 1)) * p.Hq + hr;
    const bool to_resp = is_resp && p.chain_mode != 2;
    float* o_dst = (to_resp ? p.o_resp : p.o_out) + out_row * p.dv_total + dvh * DV;
    float* lse_dst = (to_resp ? p.lse_resp : p.lse_out) + out_row;
    if (dvh != 0 && it.chained) lse_dst = p.lse_aux + out_row;     // the second O half's chain keeps its own copy of l
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    if (n_tiles > 0) {
      const int64_t lim = is_resp ? (int64_t)min(t, p.R - 1) : tokens - 1;
      const float thresh = kRescaleLog2 / p.scale_log2;
      const uint32_t p_remote[2] = {mapa_u32(smem_u32(&p_full[0]), 0), mapa_u32(smem_u32(&p_full[1]), 0)};
      for (int i = 0; i < n_tiles && ok; ++i) {
        const uint32_t ts = tmem_s0 + (i & 1) * 128 + lane_sel;
        ok = LS_TWAIT(tw0, mbar_wait_warp(&s_full[i & 1], (i >> 1) & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        uint32_t sr[128];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(ts + c * 32, sr + c * 32);
#pragma unroll
        for (int c = 0; c < 4; ++c) tc_wait_ld32(sr + c * 32);
        float* s = reinterpret_cast<float*>(sr);
        const int key0 = i * 128;
        if (__any_sync(0xffffffffu, (int64_t)key0 + 127 > lim)) {
#pragma unroll
          for (int j = 0; j < 128; ++j)
            if ((int64_t)key0 + j > lim) s[j] = -INFINITY;
        }
        float mx0 = s[0], mx1 = s[1], mx2 = s[2], mx3 = s[3];
#pragma unroll
        for (int j = 4; j < 128; j += 4) {
          mx0 = fmaxf(mx0, s[j]);
          mx1 = fmaxf(mx1, s[j + 1]);
          mx2 = fmaxf(mx2, s[j + 2]);
          mx3 = fmaxf(mx3, s[j + 3]);
        }
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        if (i == 0) {
          m_ref = (mx == -INFINITY) ? 0.f : mx;
        } else if (__any_sync(0xffffffffu, row_ok && mx > m_ref + thresh)) {   // (rows outside the tile hold stale bytes: they must not steer the warp)
          // rare: raise the reference maximum and rescale the running sum and O (this CTA's rows)
          ok = mbar_wait_warp(pv_done, (i - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const float m_new = fmaxf(m_ref, mx);
          const float f = ex2((m_ref - m_new) * p.scale_log2);
          m_ref = m_new;
          l *= f;
#pragma unroll 1
          for (int c = 0; c < DV; c += 32) {
            uint32_t o[32];
            tmem_ld32(tmem_o + lane_sel + c, o);
            tc_wait_ld32(o);
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * f);
            tmem_st32(tmem_o + lane_sel + c, o);
          }
          tc_wait_st();
        }
        const float neg_m = -m_ref * p.scale_log2;
        uint32_t pk[64];
        float l0 = 0.f, l1 = 0.f;
#pragma unroll
        for (int j = 0; j < 128; j += 2) {
          const float p0 = ex2(fmaf(s[j], p.scale_log2, neg_m));
          const float p1 = ex2(fmaf(s[j + 1], p.scale_log2, neg_m));
          l0 += p0;
          l1 += p1;
          pk[j >> 1] = pack_bf16(p0, p1);
        }
        l += l0 + l1;
        tmem_st32(ts, pk);
        tmem_st32(ts + 32, pk + 32);
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(p_remote[i & 1]);   // one arrival per warp, at the even CTA
      }
      if (threadIdx.x == 64) {
        LS_TDUMP(16, tw0);
        LS_TDUMP(18, clock64() - t_begin);
      }
      if (ok) ok = mbar_wait_warp(o_final, 0, abort_flag);
      if (ok) tc_fence_after();
    }
    // ---- epilogue: store this partial, or fold it into the running value of its chain
    const bool chained = it.chained && tile_ok;
    int* counter = chained ? p.ctl + kChainHeaderInts + fwd_chain_index(p, it, qtile) * NDV + dvh : nullptr;
    const bool fold = chained && !it.first;
    if (ok && fold) ok = __all_sync(0xffffffffu, chain_wait(counter, it.link, p.ctl, abort_flag));
    if (ok)
      fwd_store_row<DV>(tmem_o + lane_sel, n_tiles > 0, l, m_ref * p.scale, fold, o_dst, lse_dst,
                        dvh == 0 || chained,
                        (it.last && p.o_bf16) ? p.o_bf16 + out_row * p.dv_total + dvh * DV : nullptr, row_ok, chained,
                        chained && (p.chain_mode == 2 ? it.last : it.link == p.fine - 1));
    if (chained) {
      const bool all_ok = bar_and(2, 128, ok);     // every row of the tile is written
      if (row == 0 && all_ok) chain_publish(counter, it.link + 1);
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
    if (p.ctl) st_relaxed_gpu(p.ctl + 1, 1);    // ends every other chain wait of this launch
  }
}

template <int DK, int NDV>
static ls_status_t launch_fwd2(const FwdParams& prm, int64_t grid, cudaStream_t st) {
  using C = Fwd2Cfg<DK>;
  static bool configured[64] = {};
  grid *= NDV;
  if (grid > INT32_MAX) return LS_ERR_UNSUPPORTED_SHAPE;
  const ls_status_t cs = configure_smem(fwd2_kernel<DK, NDV>, C::SMEM_BYTES, configured);
  if (cs != LS_OK) return cs;
  profile_begin(LS_KERNEL_FWD, st);
  fwd2_kernel<DK, NDV><<<(int)grid, kFwdThreads, C::SMEM_BYTES, st>>>(prm);
  profile_end(LS_KERNEL_FWD, st);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

template <int DK, int DVT, int NDV>
static ls_status_t launch_fwd(const FwdParams& prm, int64_t grid, cudaStream_t st) {
  using C = FwdCfg<DK, DVT>;
  static bool configured[64] = {};
  if (grid * NDV > INT32_MAX) return LS_ERR_UNSUPPORTED_SHAPE;
  const ls_status_t cs = configure_smem(fwd_kernel<DK, DVT, NDV>, C::SMEM_BYTES, configured);
  if (cs != LS_OK) return cs;
  profile_begin(LS_KERNEL_FWD, st);
  fwd_kernel<DK, DVT, NDV><<<(int)(grid * NDV), kFwdThreads, C::SMEM_BYTES, st>>>(prm);
  profile_end(LS_KERNEL_FWD, st);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

// Shape facts shared by the entry points.
struct FwdShape {
  int R, Hq, Hkv, g, dk, dv, nq_tiles, ndv;
  RowTiling rt;
  bool mla, packed;
};
static FwdShape fwd_shape(const ls_pages* h, const ls_attn_params_t* prm) {
  FwdShape f;
  const ls_pages_desc_t& d = h->desc;
  f.R = prm->R;
  f.Hq = prm->num_q_heads;
  f.Hkv = d.num_kv_heads;
  f.g = f.Hq / f.Hkv;
  f.dk = d.dim_k;
  f.dv = d.dim_v;
  f.mla = d.dim_k == 576;
  f.rt = row_tiling(f.R, f.g, 128);            // short response: rows of several heads share a Q tile
  f.packed = f.rt.packed;
  f.nq_tiles = f.rt.nq_tiles;
  f.ndv = f.mla ? 2 : 1;
  return f;
}
// bytes of hand-over control words for `chains` chains, rounded to 16
static size_t ctl_bytes(int64_t chains) { return (size_t)((kChainHeaderInts + chains) * sizeof(int) + 15) & ~(size_t)15; }

// mode: 0 / 1 = (S+1) partials (1 when shards are walked as sub-shards), 2 = composed output.
static ls_status_t run_forward(const ls_pages* h, const ls_attn_params_t* prm, int mode, const void* q,
                               const void* k_resp, const void* v_resp, float* o_out, float* lse_out, float* o_resp,
                               float* lse_resp, void* o_bf16, void* workspace, int32_t* status_dev,
                               cudaStream_t cs) {
  const ls_pages_desc_t& d = h->desc;
  const FwdShape f = fwd_shape(h, prm);
  FwdParams P;
  const int R = f.R, Hq = f.Hq, Hkv = f.Hkv;
  const int kslabs = d.dim_k == 256 ? 2 : 1;
  const int dvt = f.mla ? 256 : d.dim_v;                    // O channels per CTA
  const int vkeys = (d.dim_k == 256 ? 32768 : 16384) / (dvt * 2);
  const bool small_pages = d.page_size == 64;
  // CTA pairs share every key tile between two Q tiles; a short response whose KV group is ONE packed tile
  // streams K/V once on the single-CTA kernel
  const bool pair = (d.dim_k == 256 || f.mla) && !(f.packed && f.nq_tiles == 1);
  if (prm->flags & LS_FLAG_NO_RESPONSE_BLOCK) k_resp = v_resp = q;   // the response maps are encoded but never used
  ls_status_t st = encode_map_rows(&P.q_map, q, d.dim_k, R, Hq, f.rt.bt, f.rt.bh);
  if (pair) {
    if (st == LS_OK)
      st = encode_map5(&P.rk2, k_resp, d.dim_k, R, Hkv, 1, (int64_t)Hkv * d.dim_k, d.dim_k, (int64_t)R * Hkv * d.dim_k, 64, 2);
    if (st == LS_OK)
      st = encode_map5(&P.rv2, v_resp, d.dim_v, R, Hkv, 1, (int64_t)Hkv * d.dim_v, d.dim_v, (int64_t)R * Hkv * d.dim_v, 64, 2);
    if (f.mla) {
      if (st == LS_OK)
        st = encode_map5(&P.rk1, k_resp, d.dim_k, R, Hkv, 1, (int64_t)Hkv * d.dim_k, d.dim_k, (int64_t)R * Hkv * d.dim_k, 64, 1);
      if (st == LS_OK) st = pool_map(&P.pk1, h, 0, 64, 1, false);
      if (st == LS_OK) st = pool_map(&P.pk1_tail, h, 0, 64, 1, true);
    }
    if (st == LS_OK) st = pool_map(&P.pk2, h, 0, 64, 2, false);
    if (st == LS_OK) st = pool_map(&P.pk2_tail, h, 0, 64, 2, true);
    if (st == LS_OK) st = pool_map(&P.pv2, h, 1, 64, 2, false);
    if (st == LS_OK) st = pool_map(&P.pv2_tail, h, 1, 64, 2, true);
  } else {
    if (st == LS_OK)
      st = encode_map5(&P.kr_map, k_resp, d.dim_k, R, Hkv, 1, (int64_t)Hkv * d.dim_k, d.dim_k,
                       (int64_t)R * Hkv * d.dim_k, 128, kslabs);
    if (st == LS_OK)
      st = encode_map5(&P.vr_map, v_resp, d.dim_v, R, Hkv, 1, (int64_t)Hkv * d.dim_v, d.dim_v,
                       (int64_t)R * Hkv * d.dim_v, vkeys, dvt / 64);
    const int kbox = small_pages ? 64 : 128, kgroups = small_pages ? 1 : kslabs;
    if (st == LS_OK) st = pool_map(&P.k_map, h, 0, kbox, kgroups, false);
    if (st == LS_OK) st = pool_map(&P.k_tail_map, h, 0, kbox, kgroups, true);
    if (st == LS_OK) st = pool_map(&P.v_map, h, 1, vkeys, dvt / 64, false);
    if (st == LS_OK) st = pool_map(&P.v_tail_map, h, 1, vkeys, dvt / 64, true);
  }
  if (st != LS_OK) return st;
  P.part_pages = h->d_part_pages;
  P.part_page_offset = h->d_part_page_offset;
  P.part_tail_slot = h->d_part_tail_slot;
  P.part_tokens = h->d_part_tokens;
  const int parts = h->num_parts();
  P.o_out = o_out;
  P.lse_out = lse_out;
  P.o_resp = o_resp;
  P.lse_resp = lse_resp;
  P.o_bf16 = static_cast<__nv_bfloat16*>(o_bf16);
  P.status = status_dev;
  P.timing = g_timing_buffer;
  P.R = R;
  P.Hq = Hq;
  P.Hkv = Hkv;
  P.g = f.g;
  P.parts = parts;
  P.pg_shift = pg_shift_of(d.page_size);
  P.nq_tiles = f.nq_tiles;
  P.bt = f.rt.bt;
  P.bh = f.rt.bh;
  P.tiles_tok = f.rt.tiles_tok;
  P.q_bytes = (d.dim_k / 64) * f.rt.bt * f.rt.bh * 128;
  P.num_phys_pages = (int)std::min<int64_t>(d.num_phys_pages, INT32_MAX);
  P.dv_total = d.dim_v;
  P.chain_mode = mode;
  P.no_resp = (prm->flags & LS_FLAG_NO_RESPONSE_BLOCK) ? 1 : 0;
  P.fine = h->fine;
  P.ablate = prm->flags & LS_DBG_ABLATE_MASK;
  P.scale = prm->scale;
  P.scale_log2 = prm->scale * 1.4426950408889634f;
  // hand-over control words (and the second running l of the two-tile shape) at the workspace's start
  P.ctl = nullptr;
  P.lse_aux = nullptr;
  if (mode != 0) {
    const int64_t groups = mode == 2 ? Hkv : (int64_t)Hkv * d.num_shards;
    const size_t cb = ctl_bytes(groups * f.nq_tiles * f.ndv);
    P.ctl = static_cast<int*>(workspace);
    P.lse_aux = reinterpret_cast<float*>(static_cast<char*>(workspace) + cb);
    if (cudaMemsetAsync(workspace, 0, cb, cs) != cudaSuccess) return LS_ERR_CUDA;
  }
  if (pair) {
    const int64_t grid2 = (int64_t)Hkv * (parts + 1) * ((f.nq_tiles + 1) / 2) * 2;
    return f.mla ? launch_fwd2<576, 2>(P, grid2, cs) : launch_fwd2<256, 1>(P, grid2, cs);
  }
  const int64_t grid = (int64_t)Hkv * (parts + 1) * f.nq_tiles;
  return f.mla ? launch_fwd<576, 256, 2>(P, grid, cs)
               : d.dim_k == 128 ? launch_fwd<128, 128, 1>(P, grid, cs) : launch_fwd<256, 256, 1>(P, grid, cs);
}

static ls_status_t check_forward_args(const ls_pages* h, const ls_attn_params_t* prm, const void* q,
                                      const void* k_resp, const void* v_resp) {
  ls_status_t st = check_handle(h, prm);
  if (st != LS_OK) return st;
  const bool no_resp = (prm->flags & LS_FLAG_NO_RESPONSE_BLOCK) != 0;
  if (!q || (!no_resp && (!k_resp || !v_resp))) return LS_ERR_INVALID_ARG;
  const ls_pages_desc_t& d = h->desc;
  if (prm->R < 1 || prm->num_q_heads < 1 || prm->num_q_heads % d.num_kv_heads != 0) return LS_ERR_INVALID_ARG;
  if (!(prm->scale > 0.f)) return LS_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_resp) || !aligned16(v_resp)) return LS_ERR_ALIGNMENT;
  return LS_OK;
}

}  // namespace ls

extern "C" size_t ls_replay_attn_workspace_bytes(const ls_pages_t* h, const ls_attn_params_t* prm, int which) {
  if (!h || !prm || prm->R < 1 || prm->num_q_heads < 1 || prm->num_q_heads % h->desc.num_kv_heads != 0) return 0;
  const ls::FwdShape f = ls::fwd_shape(h, prm);
  const size_t rows = (size_t)f.R * f.Hq;
  const ls_pages_desc_t& d = h->desc;
  if (which == LS_WORKSPACE_FWD) {
    // nothing unless shards are walked as sub-shards: then one hand-over counter per (KV head, shard, Q tile)
    if (h->fine == 1) return 0;
    return ls::ctl_bytes((int64_t)f.Hkv * d.num_shards * f.nq_tiles * f.ndv) +
           (f.mla ? (size_t)d.num_shards * rows * sizeof(float) : 0);
  }
  if (which == LS_WORKSPACE_FWD_MERGED)
    return ls::ctl_bytes((int64_t)f.Hkv * f.nq_tiles * f.ndv) + (f.mla ? rows * sizeof(float) : 0);
  if (which != LS_WORKSPACE_BWD) return 0;
  // backward: Delta (fp32) + hand-over counters + the fp32 dQ that the partials are summed into
  const bool mla_fast = f.mla && ls::mla_dq_fast(h);
  int64_t chains = (int64_t)f.Hkv * f.g * ((f.R + 127) / 128);
  if (mla_fast) chains = std::max(chains, ls::mla_dq_blocks(h, f.R, f.Hq));     // its row blocks are 64 rows
  size_t head = ((rows * sizeof(float) + 15) & ~(size_t)15) + ls::ctl_bytes(chains);
  if (f.mla) {         // head ranges of the response dK / dV, each with an fp32 sum
    const int hsplit = ls::mla_kv_hsplit(h, f.R, f.Hq);
    if (hsplit > 1) head += (size_t)hsplit * f.R * f.Hkv * d.dim_k * sizeof(float);
  }
  if (f.mla && !mla_fast)     // 576/512 with a separate V pool: one fp32 dQ per partial
    return head + (size_t)(h->num_parts() + 1) * rows * d.dim_k * sizeof(float);
  // (short responses of the aliased 576/512 shape spread the parts over several CTA pairs per row block,
  // each with an fp32 sum of its own)
  size_t partials = 0;
  if (mla_fast) {
    const ls::MlaDqSplit sp = ls::mla_dq_split(h, f.R, f.Hq);
    if (sp.count > 1 && !sp.chain) partials = (size_t)sp.count;
  } else if (!f.mla && f.packed && f.nq_tiles == 1) {
    // a short response whose KV group is one Q tile: one fp32 sum per CTA, then a reduce (no chain of
    // folds at the end of the launch)
    partials = (size_t)ls::dq1_ranges(f.Hkv, d.prefix_len);
  }
  return head + (1 + partials) * rows * d.dim_k * sizeof(float);
}

extern "C" ls_status_t ls_replay_attn_fwd(const ls_pages_t* h, const ls_attn_params_t* prm, const void* q,
                                          const void* k_resp, const void* v_resp, float* o_part, float* lse_part,
                                          void* workspace, size_t workspace_bytes, int32_t* status_dev,
                                          void* stream) {
  ls_status_t st = ls::check_forward_args(h, prm, q, k_resp, v_resp);
  if (st != LS_OK) return st;
  if (!o_part || !lse_part) return LS_ERR_INVALID_ARG;
  if (!ls::aligned16(o_part)) return LS_ERR_ALIGNMENT;
  if (!h->suffix_blocks.empty()) return LS_ERR_INVALID_ARG;     // per-shard partials describe the prefix only
  const size_t need = ls_replay_attn_workspace_bytes(h, prm, LS_WORKSPACE_FWD);
  if (need && (!workspace || workspace_bytes < need || !ls::aligned16(workspace))) return LS_ERR_WORKSPACE;
  const int64_t rows_all = (int64_t)prm->R * prm->num_q_heads;
  const int S = h->desc.num_shards;
  return ls::run_forward(h, prm, h->fine > 1 ? 1 : 0, q, k_resp, v_resp, o_part, lse_part,
                         o_part + (size_t)S * rows_all * h->desc.dim_v, lse_part + (size_t)S * rows_all, nullptr,
                         workspace, status_dev, static_cast<cudaStream_t>(stream));
}

extern "C" ls_status_t ls_replay_attn_fwd_merged(const ls_pages_t* h, const ls_attn_params_t* prm, const void* q,
                                                 const void* k_resp, const void* v_resp, void* o_bf16, float* o_f32,
                                                 float* lse, void* workspace, size_t workspace_bytes,
                                                 int32_t* status_dev, void* stream) {
  ls_status_t st = ls::check_forward_args(h, prm, q, k_resp, v_resp);
  if (st != LS_OK) return st;
  if (!o_f32 || !lse) return LS_ERR_INVALID_ARG;
  if (!ls::aligned16(o_f32) || !ls::aligned16(o_bf16)) return LS_ERR_ALIGNMENT;
  const size_t need = ls_replay_attn_workspace_bytes(h, prm, LS_WORKSPACE_FWD_MERGED);
  if (!workspace || workspace_bytes < need || !ls::aligned16(workspace)) return LS_ERR_WORKSPACE;
  return ls::run_forward(h, prm, 2, q, k_resp, v_resp, o_f32, lse, nullptr, nullptr, o_bf16, workspace, status_dev,
                         static_cast<cudaStream_t>(stream));
}
