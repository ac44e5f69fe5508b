// Query gradient over the prefix for the shared-latent shape whose value is the first 512
// channels of the 576-channel key page (Sec. "GLM page payloads"; dense form):
//   dQ_th = scale * sum_j p_tj (dO_th . v_j - Delta_th) k_j,   p_tj = exp(scale q_th . k_j - LSE_th).
//
// The products are formed TRANSPOSED, keys on the tensor core's M side, so that a CTA can
// keep only 64 rows (Q 72 KB + dO 64 KB) and still fill every 128-row instruction:
//   [S^T | T^T] (128 keys x 128) = K_c (128 keys x 64 ch)  x  [Q_c ; dO_c]^T   c = 0..7
//        Q and dO of the same 64-channel group lie back to back in shared memory, so one
//        128x128x16 instruction yields 64 columns of S^T and 64 of T^T (V = K[:, :512]);
//   S^T += K_8 x Q_8^T  (rope channels, N = 64);
//   E^T  = p (T^T - Delta) : one thread per key, written to shared memory as bf16, keys x 64 rows;
//   dQ^T (576 ch x 64 rows) += K^T (128 ch x 16 keys, MN-major view of the same slabs) x E^T.
// The 576 x 64 fp32 accumulator is five 128-lane tiles of 64 TMEM columns (320 columns; the
// upper half of the fifth is unused), [S^T | T^T] one buffer of 128 columns.  Every CTA walks
// ALL prefix partials in order and keeps accumulating, which is Eq. qwen-dq-reduce carried out
// in the accumulator; the causal response block (whose V is a separate tensor) arrives as an
// fp32 partial from the generic kernel and is added in the epilogue, which writes bf16 dQ.
//
// Every key tile streams through shared memory twice, in 16 KB slots of two small rings: as
// nine K-major slabs (128 keys x one channel group) for [S^T | T^T], and as ten MN-major
// slots (64 keys x two channel groups; the missing partner of the rope group reads as zeros)
// for dQ^T.  Two threads issue the two kinds of products, so that dQ^T of tile i overlaps
// [S^T | T^T] of tile i + 2 while the key threads work on tile i + 1.
#include <cuda_bf16.h>

#include <algorithm>

#include "ls_internal.h"
#include "ls_sm100.cuh"

namespace ls {

struct MlaDqParams {
  CUtensorMap q_map, do_map;         // dense rows: box 64 ch x 64 tokens
  CUtensorMap k_map, k_tail;         // prefix pool key page: box 64 ch x 64 tokens
  CUtensorMap k2_map, k2_tail;       // the same with two channel groups per box
  const int32_t* shard_phys_pages;
  const int32_t* shard_page_offset;
  const int32_t* shard_tail_slot;
  const int64_t* shard_tokens;
  const float* lse;
  const float* delta;
  const float* dq_resp;              // [R, Hq, 576] fp32, unscaled: the response block's part (NULL: none)
  __nv_bfloat16* dq;                 // [R, Hq, 576]
  int32_t* status;
  long long* timing;   // diagnostic builds only
  int R, Hq, g, nparts, pg_shift, num_phys_pages;
  // Row blocks of a KV group (RowTiling with 64-row tiles): block q covers bt tokens from (q % tiles_tok) * bt
  // of bh heads from (q / tiles_tok) * bh; its row r is head r / bt, token r % bt.  Long responses: 64 x 1.
  int bt, bh, tiles_tok, nq_tiles;
  int qdo_bytes;   // bytes the Q and dO loads deliver
  int nsplit;      // CTAs per row block, each walking a contiguous range of the parts; with more than one
                   // the fp32 sums go to dq_split [nsplit, R, Hq, 576] and a reduce kernel finishes
  float* dq_split;
  int ablate;   // diagnostic builds only: 1 = no key loads, 2 = no tensor-core instructions
  float scale, scale_log2;
};

// Build with -DLS_TIMING to make CTA 0 write per-role cycle counts (time spent in each kind
// of wait, and in total) into the buffer given to ls_debug_timing_buffer; a profiling aid.
#ifdef LS_TIMING
#define LS_TQWAIT(acc, expr) ([&] { const long long t0_ = clock64(); const bool r_ = (expr); (acc) += clock64() - t0_; return r_; }())
#define LS_TQDUMP(slot, val) do { if (blockIdx.x == 0 && p.timing) p.timing[(slot)] = (val); } while (0)
#define LS_TQABLATE(bit) (p.ablate & (bit))
#else
#define LS_TQWAIT(acc, expr) (expr)
#define LS_TQDUMP(slot, val) do { } while (0)
#define LS_TQABLATE(bit) false
#endif

constexpr int kTqThreads = 224;   // producer, [S^T|T^T] issuer, 4 warps of key threads, dQ^T issuer
constexpr int kTqSlab = 16384;                 // 128 keys x 128 B
constexpr int kTqRing = 4;                   // ring slots of 16 KB:
constexpr int kTqStSlots = 2;                //   [S^T | T^T] slabs
constexpr int kTqAccSlots = kTqRing - kTqStSlots;   //   dQ^T slots
constexpr int kTqRows = 64;
constexpr int kTqQdo = 8 * 16384 + 8192;       // [Q_c | dO_c] c = 0..7, then Q_8
constexpr int kTqSmem = 1024 + kTqQdo + kTqRing * kTqSlab + kTqSlab + 512 + 256;
constexpr float kLog2eTq = 1.4426950408889634f;

__global__ void __launch_bounds__(kTqThreads, 1) bwd_mla_dq_kernel(const __grid_constant__ MlaDqParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* qdo = smem;
  uint8_t* ring = qdo + kTqQdo;
  uint8_t* e_smem = ring + kTqRing * kTqSlab;
  float2* rowp = reinterpret_cast<float2*>(e_smem + kTqSlab);     // (LSE * log2 e, Delta) of the 64 rows
  uint64_t* bars = reinterpret_cast<uint64_t*>(e_smem + kTqSlab + 512);
  uint64_t* a_full = bars;
  uint64_t* full = bars + 1;
  uint64_t* empty = full + kTqRing;
  uint64_t* st_full = empty + kTqRing;
  uint64_t* s_read = st_full + 1;
  uint64_t* e_full = s_read + 1;
  uint64_t* e_free = e_full + 1;
  uint64_t* acc_final = e_free + 1;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_final + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  long long tw0 = 0, tw1 = 0, tw2 = 0, tw3 = 0;   // wait-time accumulators (only used with LS_TIMING)
  const long long t_begin = clock64();
  // work item: row block (fastest, so that the CTAs in flight share the same keys), range of parts, KV head
  const int qtile = blockIdx.x % p.nq_tiles;
  const int split = (blockIdx.x / p.nq_tiles) % p.nsplit;
  const int kvh = blockIdx.x / (p.nq_tiles * p.nsplit);
  const int h = kvh * p.g + (qtile / p.tiles_tok) * p.bh;     // first head and token of the block
  const int row0 = (qtile % p.tiles_tok) * p.bt;
  // the parts this CTA walks: all of them, or (several CTAs per row block) a contiguous range
  const int part_lo = (int)((long long)split * p.nparts / p.nsplit);
  const int part_hi = (int)((long long)(split + 1) * p.nparts / p.nsplit);

  // key tiles of 128 over those parts (every role walks the same list)
  int total_tiles = 0;
  for (int r = part_lo; r < part_hi; ++r) total_tiles += (int)((p.shard_tokens[r] + 127) >> 7);

  if (threadIdx.x == 0) {
    mbar_init(a_full, 1);
    for (int i = 0; i < kTqRing; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    mbar_init(st_full, 1);
    mbar_init(s_read, 128);
    mbar_init(e_full, 128);
    mbar_init(e_free, 1);
    mbar_init(acc_final, 1);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (threadIdx.x >= 64 && threadIdx.x < 64 + kTqRows) {
    const int t = threadIdx.x - 64;
    const int hj = t / p.bt;
    const size_t ri = (size_t)min(row0 + t - hj * p.bt, p.R - 1) * p.Hq + min(h + hj, p.Hq - 1);
    rowp[t] = make_float2(p.lse[ri] * kLog2eTq, p.delta[ri]);
  }
  if (warp == 1) {
    tmem_alloc(tmem_holder, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  const uint32_t tmem_acc = tmem_base;          // 5 x 64 columns
  const uint32_t tmem_st = tmem_base + 320;     // S^T [0,64) | T^T [64,128)

  if (warp == 0) {
    // =========================================================== producer (one thread)
    // Two rings: slots [0, kTqStSlots) carry K-major slabs (128 keys x one channel group, two
    // 64-token boxes) for [S^T | T^T]; the rest carry MN-major slots (64 keys x two channel
    // groups, one box) for dQ^T.  The dQ^T loads of tile i are interleaved one to one with the
    // [S^T | T^T] loads of tile i + 2, the order in which the two issuers consume them.
    if (lane == 0 && total_tiles > 0) {
      mbar_arrive_expect_tx(a_full, p.qdo_bytes);
      for (int c = 0; c < 9; ++c) tma_load_5d(qdo + c * 16384, &p.q_map, a_full, 0, row0, c, h, 0);
      for (int c = 0; c < 8; ++c) tma_load_5d(qdo + c * 16384 + 8192, &p.do_map, a_full, 0, row0, c, h, 0);

      const int pg_mask = (1 << p.pg_shift) - 1;
      bool ok = true;
      // A walk over the key tiles of all partials; everything that needs global memory (the two
      // 64-token boxes of a tile) is resolved once per tile.
      struct Walk {
        int part, tile, c_off, c_pages, c_tail, c_tiles;
        int page[2], tok[2];
        bool tail[2];
      };
      auto open_part = [&](Walk& w, int r) {
        w.part = r;
        w.c_off = p.shard_page_offset[r];
        w.c_pages = p.shard_page_offset[r + 1] - w.c_off;
        w.c_tail = p.shard_tail_slot[r];
        w.c_tiles = (int)((p.shard_tokens[r] + 127) >> 7);
      };
      auto next_tile = [&](Walk& w) {
        ++w.tile;
        while (w.part < part_hi && w.tile >= w.c_tiles) {
          w.tile = 0;
          if (w.part + 1 < part_hi) open_part(w, w.part + 1); else ++w.part;
        }
        if (w.part >= part_hi) return;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int tok = w.tile * 128 + half * 64;
          const int ps = tok >> p.pg_shift;
          // past the part's last page: a coordinate beyond the pool, where TMA fills zeros (the bytes of
          // an arbitrary page could be NaN patterns, and 0 * NaN would poison dQ^T)
          w.page[half] = ps < w.c_pages ? __ldg(p.shard_phys_pages + w.c_off + ps) : p.num_phys_pages;
          w.tok[half] = tok & pg_mask;
          w.tail[half] = ps == w.c_tail;
        }
      };
      uint32_t s_seq = 0, a_seq = 0, issued_s = 0, issued_a = 0;
      auto load_st = [&](const Walk& w, int c) {          // channel group c of the tile
        const uint32_t slot = s_seq % kTqStSlots, lap = s_seq / kTqStSlots;
        ok = ok && LS_TQWAIT(tw0, mbar_wait(&empty[slot], (lap & 1) ^ 1, abort_flag));
        if (ok) {
          uint8_t* dst = ring + slot * kTqSlab;
          if (LS_TQABLATE(1)) {
            mbar_arrive(&full[slot]);
          } else {
            mbar_arrive_expect_tx(&full[slot], kTqSlab);
            tma_load_5d(dst, w.tail[0] ? &p.k_tail : &p.k_map, &full[slot], 0, w.tok[0], c, kvh, w.page[0]);
            tma_load_5d(dst + 8192, w.tail[1] ? &p.k_tail : &p.k_map, &full[slot], 0, w.tok[1], c, kvh, w.page[1]);
          }
          ++issued_s;
        }
        ++s_seq;
      };
      auto load_acc = [&](const Walk& w, int k) {         // k = half * 5 + channel-group pair
        const uint32_t slot = kTqStSlots + a_seq % kTqAccSlots, lap = a_seq / kTqAccSlots;
        ok = ok && LS_TQWAIT(tw1, mbar_wait(&empty[slot], (lap & 1) ^ 1, abort_flag));
        if (ok) {
          const int half = k >= 5 ? 1 : 0, m = k - half * 5;
          if (LS_TQABLATE(1)) {
            mbar_arrive(&full[slot]);
          } else {
            mbar_arrive_expect_tx(&full[slot], kTqSlab);
            tma_load_5d(ring + slot * kTqSlab, w.tail[half] ? &p.k2_tail : &p.k2_map, &full[slot], 0, w.tok[half],
                        2 * m, kvh, w.page[half]);
          }
          ++issued_a;
        }
        ++a_seq;
      };
      Walk ws, wa;
      ws.tile = -1;
      open_part(ws, part_lo);
      wa = ws;
      next_tile(ws);
#pragma unroll 1
      for (int c = 0; c < 9; ++c) load_st(ws, c);          // tile 0
      if (total_tiles > 1) {
        next_tile(ws);
#pragma unroll 1
        for (int c = 0; c < 9; ++c) load_st(ws, c);        // tile 1
      }
      for (int i = 0; i < total_tiles && ok; ++i) {
        const bool has_st = i + 2 < total_tiles;
        if (has_st) next_tile(ws);
        next_tile(wa);
#pragma unroll
        for (int k = 0; k < 10; ++k) {
          if (has_st && k < 9) load_st(ws, k);
          load_acc(wa, k);
        }
      }
      LS_TQDUMP(0, tw0);
      LS_TQDUMP(2, tw1);
      LS_TQDUMP(1, clock64() - t_begin);
      if (*abort_flag) {   // aborted: wait (bounded) for the copies already started
        for (int s = 0; s < kTqRing; ++s) {
          const bool st_ring = s < kTqStSlots;
          const uint32_t n = st_ring ? issued_s : issued_a, per = st_ring ? kTqStSlots : kTqAccSlots;
          const uint32_t idx = st_ring ? s : s - kTqStSlots;
          if (n <= idx) continue;
          const uint32_t last_lap = (n - 1 - idx) / per;
          const uint64_t t_start = globaltimer_ns();
          while (!mbar_try_wait(&full[s], last_lap & 1, 1000) && globaltimer_ns() - t_start < 100000000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // =========================================================== [S^T | T^T] issuer (one thread)
    // The two kinds of products are issued by two threads (this one and one of warp 6), each
    // from its own ring: they write disjoint TMEM columns and each thread's own instructions
    // stay in order, so the per-slot bookkeeping of one overlaps the other's.
    if (lane == 0 && total_tiles > 0) {
      constexpr uint32_t idesc_st = make_idesc(128, 128, 0, 0);
      constexpr uint32_t idesc_rope = make_idesc(128, 64, 0, 0);
      constexpr uint32_t hi = sdesc_hi(1024);
      const uint32_t qdo_lo = sdesc_lo(smem_u32(qdo), 16);
      const uint32_t ring_k_lo = sdesc_lo(smem_u32(ring), 16);          // K-major: 128 keys x 64 channels
      bool ok = mbar_wait(a_full, 0, abort_flag);
      uint32_t seq = 0;
      for (int i = 0; i < total_tiles && ok; ++i) {
        if (i > 0) {
          ok = LS_TQWAIT(tw2, mbar_wait(s_read, (i - 1) & 1, abort_flag));   // tile i - 1 is in registers
          if (!ok) break;
          tc_fence_after();
        }
#pragma unroll
        for (int c = 0; c < 9; ++c) {
          const uint32_t slot = seq % kTqStSlots, lap = seq / kTqStSlots;
          ok = ok && LS_TQWAIT(tw0, mbar_wait(&full[slot], lap & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_lo = ring_k_lo + slot * (kTqSlab >> 4);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            if (!LS_TQABLATE(2))
              mma_ss(tmem_st, sdesc(a_lo + ((k * 32) >> 4), hi), sdesc(qdo_lo + ((c * 16384 + k * 32) >> 4), hi),
                     c < 8 ? idesc_st : idesc_rope, (c | k) != 0);
          mma_commit(&empty[slot]);
          ++seq;
        }
        if (!ok) break;
        mma_commit(st_full);
      }
      LS_TQDUMP(8, tw0);
      LS_TQDUMP(10, tw2);
      LS_TQDUMP(12, clock64() - t_begin);
    }
  } else if (warp == 6) {
    // =========================================================== dQ^T issuer (one thread)
    if (lane == 0 && total_tiles > 0) {
      constexpr uint32_t idesc_acc = make_idesc(128, 64, 1, 1);
      constexpr uint32_t hi = sdesc_hi(1024);
      const uint32_t ring_m_lo = sdesc_lo(smem_u32(ring), 8192);        // MN-major: 64 keys x two channel groups
      const uint32_t e_lo = sdesc_lo(smem_u32(e_smem), 16);             // MN-major: keys x 64 rows
      bool ok = true;
      uint32_t seq = 0;
      for (int i = 0; i < total_tiles && ok; ++i) {
        ok = LS_TQWAIT(tw3, mbar_wait(e_full, i & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < 10; ++k) {
          const int half = k >= 5 ? 1 : 0, m = k - half * 5;
          const uint32_t slot = kTqStSlots + seq % kTqAccSlots, lap = seq / kTqAccSlots;
          ok = ok && LS_TQWAIT(tw1, mbar_wait(&full[slot], lap & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_lo = ring_m_lo + slot * (kTqSlab >> 4);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            if (!LS_TQABLATE(2))
              mma_ss(tmem_acc + m * 64, sdesc(a_lo + ((kk * 2048) >> 4), hi),
                     sdesc(e_lo + ((half * 8192 + kk * 2048) >> 4), hi), idesc_acc, (i | half | kk) != 0);
          mma_commit(&empty[slot]);
          ++seq;
        }
        if (!ok) break;
        mma_commit(e_free);
        if (i == total_tiles - 1) mma_commit(acc_final);
      }
      LS_TQDUMP(9, tw1);
      LS_TQDUMP(11, tw3);
      LS_TQDUMP(13, clock64() - t_begin);
    }
  } else {
    // =========================================================== one thread per key: E^T, epilogue
    const int quad = warp & 3;
    const int key = quad * 32 + lane;                      // TMEM lane = key of the tile
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    uint8_t* e_row = e_smem + key * 128;
    const int sw = key & 7;
    if (total_tiles > 0) {
      bool ok = true;
      int part = part_lo, tile = -1;
      for (int i = 0; i < total_tiles && ok; ++i) {
        ++tile;
        while (tile >= (int)((p.shard_tokens[part] + 127) >> 7)) {
          ++part;
          tile = 0;
        }
        const bool valid = (int64_t)tile * 128 + key < p.shard_tokens[part];
        ok = LS_TQWAIT(tw0, mbar_wait(st_full, i & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        uint32_t pk[32];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t sr[32], tr[32];
          tmem_ld32(tmem_st + lane_sel + half * 32, sr);
          tmem_ld32(tmem_st + lane_sel + 64 + half * 32, tr);
          tc_wait_ld32(sr);
          tc_wait_ld32(tr);
          if (half == 1) {          // the whole buffer is in registers: the next tile may overwrite it
            tc_fence_before();
            mbar_arrive(s_read);
          }
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            const float4 rp = *reinterpret_cast<const float4*>(rowp + half * 32 + j);   // two rows
            const float p0 = ex2(fmaf(__uint_as_float(sr[j]), p.scale_log2, -rp.x));
            const float p1 = ex2(fmaf(__uint_as_float(sr[j + 1]), p.scale_log2, -rp.z));
            pk[half * 16 + (j >> 1)] =
                pack_bf16(p0 * (__uint_as_float(tr[j]) - rp.y), p1 * (__uint_as_float(tr[j + 1]) - rp.w));
          }
        }
        if (!valid) {
#pragma unroll
          for (int j = 0; j < 32; ++j) pk[j] = 0u;
        }
        if (i > 0) {
          ok = LS_TQWAIT(tw1, mbar_wait(e_free, (i - 1) & 1, abort_flag));   // the previous tile's dQ^T instructions have read E^T
          if (!ok) break;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
          *reinterpret_cast<uint4*>(e_row + ((j ^ sw) << 4)) =
              make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
        fence_proxy_async();
        mbar_arrive(e_full);
      }
      if (threadIdx.x == 64) {
        LS_TQDUMP(16, tw0);
        LS_TQDUMP(17, tw1);
        LS_TQDUMP(18, clock64() - t_begin);
      }
      if (ok) ok = mbar_wait(acc_final, 0, abort_flag);
      if (ok) {
        tc_fence_after();
#pragma unroll 1
        for (int m = 0; m < 5; ++m) {
          if (m == 4 && quad >= 2) break;                   // channels 576.. do not exist
          const int ch = m * 128 + key;
#pragma unroll 1
          for (int half = 0; half < 2; ++half) {
            uint32_t o[32];
            tmem_ld32(tmem_acc + lane_sel + m * 64 + half * 32, o);
            tc_wait_ld32(o);
            int hj = (half * 32) / p.bt, tk = half * 32 - hj * p.bt;   // head and token of row half * 32 + j
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int r = row0 + tk, hh = h + hj;
              if (++tk == p.bt) {
                tk = 0;
                ++hj;
              }
              if (hh - h < p.bh && r < p.R && hh < (kvh + 1) * p.g) {
                const size_t idx = ((size_t)r * p.Hq + hh) * 576 + ch;
                if (p.nsplit > 1)
                  p.dq_split[(size_t)split * p.R * p.Hq * 576 + idx] = __uint_as_float(o[j]);
                else
                  p.dq[idx] = __float2bfloat16_rn((__uint_as_float(o[j]) + (p.dq_resp ? p.dq_resp[idx] : 0.f)) * p.scale);
              }
            }
          }
        }
      }
    } else if (p.nsplit > 1) {
      // an empty range of parts still owes its (zero) partial to the reduce kernel
      for (int m = 0; m < 5; ++m) {
        if (m == 4 && quad >= 2) break;
        for (int rr = 0; rr < p.bt * p.bh; ++rr) {
          const int r = row0 + rr % p.bt, hh = h + rr / p.bt;
          if (r < p.R && hh < (kvh + 1) * p.g)
            p.dq_split[(size_t)split * p.R * p.Hq * 576 + ((size_t)r * p.Hq + hh) * 576 + m * 128 + key] = 0.f;
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

bool mla_dq_fast(const ls_pages* h) {
  const ls_pages_desc_t& d = h->desc;
  return d.dim_k == 576 && d.dim_v == 512 && d.v_aliases_k && d.prefix_len > 0;
}

int mla_dq_splits(const ls_pages* h, int R, int Hq) {
  const int Hkv = h->desc.num_kv_heads;
  const int64_t blocks = (int64_t)Hkv * row_tiling(R, Hq / Hkv, kTqRows).nq_tiles;
  if (blocks >= 148) return 1;                 // enough row blocks: every CTA walks all parts
  // few rows: the parts are spread over enough CTAs to fill the GPU twice
  return std::max(1, std::min(h->prefix_parts(), (int)((148 * 2 + blocks - 1) / blocks)));
}

// dq = scale * (sum of the split partials + the response block's partial), bf16
__global__ void mla_dq_split_reduce_kernel(const float* __restrict__ part, int nsplit, const float* __restrict__ dq_resp,
                                           int64_t n4, float scale, __nv_bfloat16* __restrict__ dq) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
    float4 acc = dq_resp ? *reinterpret_cast<const float4*>(dq_resp + i * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < nsplit; ++s) {
      const float4 v = *reinterpret_cast<const float4*>(part + ((int64_t)s * n4 + i) * 4);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    uint2 pk;
    pk.x = pack_bf16(acc.x * scale, acc.y * scale);
    pk.y = pack_bf16(acc.z * scale, acc.w * scale);
    *reinterpret_cast<uint2*>(dq + i * 4) = pk;
  }
}

// dQ (bf16, final) of the 576/512 shape with V aliasing K: prefix part in this kernel, plus
// dq_resp, the response block's unscaled fp32 part computed beforehand.
ls_status_t bwd_mla_dq(const ls_pages* h, const ls_attn_params_t* prm, const void* q, const void* d_o,
                       const float* lse, const float* delta, const float* dq_resp, float* dq_split, void* dq,
                       int32_t* status_dev, cudaStream_t cs) {
  const ls_pages_desc_t& d = h->desc;
  const int R = prm->R, Hq = prm->num_q_heads;
  MlaDqParams P;
  P.shard_phys_pages = h->d_part_pages;
  P.shard_page_offset = h->d_part_page_offset;
  P.shard_tail_slot = h->d_part_tail_slot;
  P.shard_tokens = h->d_part_tokens;
  P.lse = lse;
  P.delta = delta;
  P.dq_resp = dq_resp;
  P.dq = static_cast<__nv_bfloat16*>(dq);
  P.status = status_dev;
  P.R = R;
  P.Hq = Hq;
  P.g = Hq / d.num_kv_heads;
  P.nparts = h->prefix_parts();
  P.num_phys_pages = (int)std::min<int64_t>(d.num_phys_pages, INT32_MAX);
  P.pg_shift = pg_shift_of(d.page_size);
  P.ablate = (prm->flags & LS_DBG_ABLATE_LOADS ? 1 : 0) | (prm->flags & LS_DBG_ABLATE_MMA ? 2 : 0);
  P.timing = g_timing_buffer;
  P.scale = prm->scale;
  P.scale_log2 = prm->scale * kLog2eTq;
  // a short response packs rows of several heads of a KV group into a CTA's 64 rows
  const RowTiling rt = row_tiling(R, P.g, kTqRows);
  P.bt = rt.bt;
  P.bh = rt.bh;
  P.tiles_tok = rt.tiles_tok;
  P.nq_tiles = rt.nq_tiles;
  P.qdo_bytes = (9 + 8) * rt.bt * rt.bh * 128;
  P.nsplit = dq_split ? mla_dq_splits(h, R, Hq) : 1;     // without scratch every CTA walks all parts
  P.dq_split = dq_split;
  ls_status_t st = encode_map_rows(&P.q_map, q, 576, R, Hq, rt.bt, rt.bh);
  if (st == LS_OK) st = encode_map_rows(&P.do_map, d_o, 512, R, Hq, rt.bt, rt.bh);
  if (st == LS_OK) st = pool_map(&P.k_map, h, 0, 64, 1, false);
  if (st == LS_OK) st = pool_map(&P.k_tail, h, 0, 64, 1, true);
  if (st == LS_OK) st = pool_map(&P.k2_map, h, 0, 64, 2, false);
  if (st == LS_OK) st = pool_map(&P.k2_tail, h, 0, 64, 2, true);
  if (st != LS_OK) return st;
  static bool configured[64] = {};
  const ls_status_t cfg = configure_smem(bwd_mla_dq_kernel, kTqSmem, configured);
  if (cfg != LS_OK) return cfg;
  const int64_t grid = (int64_t)d.num_kv_heads * rt.nq_tiles * P.nsplit;
  if (grid > INT32_MAX) return LS_ERR_UNSUPPORTED_SHAPE;
  profile_begin(LS_KERNEL_BWD_DQ, cs);
  bwd_mla_dq_kernel<<<(int)grid, kTqThreads, kTqSmem, cs>>>(P);
  if (P.nsplit > 1) {
    const int64_t n4 = (int64_t)R * Hq * 576 / 4;
    mla_dq_split_reduce_kernel<<<(int)std::min<int64_t>((n4 + 255) / 256, 148 * 8), 256, 0, cs>>>(
        dq_split, P.nsplit, dq_resp, n4, prm->scale, static_cast<__nv_bfloat16*>(dq));
  }
  profile_end(LS_KERNEL_BWD_DQ, cs);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

}  // namespace ls
