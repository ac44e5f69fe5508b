// Query gradient over the prefix for the shared-latent shape whose value is the first 512
// channels of the 576-channel key page (Sec. "GLM page payloads"; dense form):
//   dQ_th = scale * sum_j p_tj (dO_th . v_j - Delta_th) k_j,   p_tj = exp(scale q_th . k_j - LSE_th).
//
// The products are formed TRANSPOSED, keys on the tensor core's M side, so that 64 rows (Q 72 KB,
// dO 64 KB) still fill every 128-row instruction, and on CTA PAIRS (cta_group::2): the even CTA
// keeps Q of the 64 rows, the odd CTA keeps dO, and a step covers 256 keys, 128 per CTA.
//   [S^T | T^T] (256 keys x 128) = K_c (this CTA's 128 keys x 64 ch) x [Q_c ; dO_c]^T   c = 0..7
//        the B operand of a pair instruction is split along N between the two CTAs, so the Q half
//        yields 64 columns of S^T and the dO half 64 columns of T^T (V = K[:, :512]) in BOTH CTAs'
//        TMEM, each for its own keys;
//   S^T += K_8 x Q_8^T  (rope channels, N = 64: each CTA contributes 32 rows of Q_8, of which both
//        hold a copy);
//   E^T  = p (T^T - Delta) : two threads per key, 32 rows each.  dQ^T is split along the channels
//        (M) between the CTAs, and its B operand E^T along the rows (N): rows 0-31 of a key go into
//        the even CTA's shared memory and rows 32-63 into the odd CTA's (st.shared::cluster), as
//        bf16 in MN-major 64-byte lines;
//   dQ^T (this CTA's 128 of 256 channels x 64 rows) += K^T (MN-major, 16 keys) x E^T, for the keys
//        of either CTA.  Channel block m = groups 4m, 4m+1 (even CTA) and 4m+2, 4m+3 (odd CTA);
//        block 2 is the 64 rope channels in the even CTA alone.
// TMEM per CTA: two [S^T | T^T] buffers of 128 columns and three accumulator tiles of 64 columns.
// Every pair walks ALL prefix partials in order and keeps accumulating, which is Eq. qwen-dq-reduce
// carried out in the accumulator; the causal response block (whose V is a separate tensor) arrives
// as an fp32 partial from the generic kernel and is added in the epilogue, which writes bf16 dQ.
//
// Every key tile streams through shared memory twice, in 16 KB slots of two rings with a producer
// thread each: K-major slabs (this CTA's 128 keys x one channel group) for [S^T | T^T], and
// MN-major slots (64 keys of either CTA's tile x two of this CTA's channel groups) for dQ^T.  Two
// threads of the even CTA issue the two kinds of products, so that dQ^T of step i overlaps
// [S^T | T^T] of step i + 1 while the key threads of both CTAs work between them; E^T and
// [S^T | T^T] are double-buffered.  What bounds it at full size is the stream itself: every 64-row
// block pulls 2.3 KB per key out of L2, and beside the resident rows only seven ring slots (112 KB
// of loads in flight per SM) fit in shared memory.
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
  // chain != 0 (many row blocks): the pairs of one range of parts run together (work items handed out by
  // ticket, range-major) so that its keys stay in L2, and the ranges' sums of a row block meet in ONE
  // running fp32 dQ, dq_acc [R, Hq, 576], in range order (ordered hand-over: ctl[0] ticket, ctl[1] abort,
  // ctl[4 + row block] completed CTAs); acc_init: dq_acc already holds the response block's partial.
  int chain, acc_init;
  int* ctl;
  float* dq_acc;
  int num_kv_heads;
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

constexpr int kTqKt = 2;                        // threads per key: each forms E^T for 64 / kTqKt of the rows
// warps: 0 K-major producer, 1 [S^T|T^T] issuer, 2 dQ^T issuer, 3 MN-major producer, then 4 * kTqKt warps of key threads
constexpr int kTqThreads = 128 + 128 * kTqKt;
static_assert(kTqKt == 2, "a key thread's rows are one CTA's half of E^T");
constexpr int kTqSlab = 16384;                 // 128 keys x 128 B
constexpr int kTqStSlots = 3;                  // ring slots of 16 KB: [S^T | T^T] slabs
constexpr int kTqAccSlots = 4;                 //                      dQ^T slots
constexpr int kTqRing = kTqStSlots + kTqAccSlots;
constexpr int kTqRows = 64;
// Row operands of a CTA: eight 8 KB slabs (64 rows x 64 channels) -- Q_c in the even CTA, dO_c in
// the odd one -- and the rope slab Q_8 of all 64 rows, placed so that the half of its rows a CTA
// contributes (rows 0-31 even, 32-63 odd) starts at the same offset kTqRope in both.
constexpr int kTqRope = 8 * 8192 + 4096;
constexpr int kTqB = kTqRope + 8192;
constexpr int kTqE = 2 * 8192;                 // E^T of the even and of the odd CTA's keys: this CTA's 32 rows of each
constexpr int kTqEBufs = 2;                    // E^T buffers: step i + 1 is written while dQ^T of step i reads
constexpr int kTqSmem = 1024 + kTqB + kTqRing * kTqSlab + kTqEBufs * kTqE + 512 + 256;
constexpr float kLog2eTq = 1.4426950408889634f;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kTqThreads, 1)
    bwd_mla_dq_kernel(const __grid_constant__ MlaDqParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* bop = smem;
  uint8_t* ring = bop + kTqB;
  uint8_t* e_smem = ring + kTqRing * kTqSlab;
  float2* rowp = reinterpret_cast<float2*>(e_smem + kTqEBufs * kTqE);        // (LSE * log2 e, Delta) of the 64 rows
  uint64_t* bars = reinterpret_cast<uint64_t*>(e_smem + kTqEBufs * kTqE + 512);
  uint64_t* a_full = bars;               // (even CTA) the row operands of both CTAs landed
  uint64_t* full = bars + 1;             // (even CTA) both CTAs' halves of a slot landed
  uint64_t* empty = full + kTqRing;      // (each CTA)
  uint64_t* st_full = empty + kTqRing;   // [2] (each CTA) one per [S^T | T^T] buffer
  uint64_t* s_read = st_full + 2;        // [2] (even CTA) 8 warp arrivals: both CTAs hold the buffer's tile in registers
  uint64_t* e_full = s_read + 2;         // [2] (even CTA) 8 warp arrivals: E^T of both CTAs' keys is written to the buffer
  uint64_t* e_free = e_full + 2;         // [2] (each CTA) one per E^T buffer
  uint64_t* acc_final = e_free + 2;      // (each CTA)
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_final + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  int* work_idx = const_cast<int*>(abort_flag) + 1;   // (even CTA) the pair's work item

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  long long tw0 = 0, tw1 = 0, tw2 = 0, tw3 = 0;   // wait-time accumulators (only used with LS_TIMING)
  const long long t_begin = clock64();
  (void)tw0; (void)tw1; (void)tw2; (void)tw3; (void)t_begin;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    // chained: work items in launch order of the pairs that ask, so that a link only waits for links some pair has started
    if (leader) *work_idx = p.chain ? atomicAdd(p.ctl, 1) : (int)(blockIdx.x >> 1);
  }
  cluster_sync_all();
  // work item of the pair: row block (fastest, so that the pairs in flight share the same keys), then
  // KV head and range of parts (chained: range slowest)
  const int work = (int)ld_shared_cluster_u32(mapa_u32(smem_u32(work_idx), 0));
  const int qtile = work % p.nq_tiles;
  const int split = p.chain ? work / (p.nq_tiles * p.num_kv_heads) : (work / p.nq_tiles) % p.nsplit;
  const int kvh = p.chain ? (work / p.nq_tiles) % p.num_kv_heads : work / (p.nq_tiles * p.nsplit);
  const int h = kvh * p.g + (qtile / p.tiles_tok) * p.bh;     // first head and token of the block
  const int row0 = (qtile % p.tiles_tok) * p.bt;
  // the parts this pair walks: all of them, or (several pairs per row block) a contiguous range
  const int part_lo = (int)((long long)split * p.nparts / p.nsplit);
  const int part_hi = (int)((long long)(split + 1) * p.nparts / p.nsplit);

  // steps of 256 keys over those parts: the even CTA takes the first 128-key tile of a step, the odd
  // CTA the second (past a part's last tile: zeros, masked).  Every role walks the same list.
  int total_steps = 0;
  for (int r = part_lo; r < part_hi; ++r) total_steps += (int)((((p.shard_tokens[r] + 127) >> 7) + 1) >> 1);

  if (threadIdx.x == 0) {
    mbar_init(a_full, 1);
    // A dQ^T slot completes only when BOTH producers have passed their wait for it (two arrivals): the
    // odd CTA loads nothing for channel block 2, and without its arrival such a slot could be filled,
    // consumed and released twice while that producer still waits for the first release.
    for (int i = 0; i < kTqRing; ++i) {
      mbar_init(&full[i], i < kTqStSlots ? 1 : 2);
      mbar_init(&empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&st_full[i], 1);
      mbar_init(&s_read[i], 8 * kTqKt);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&e_full[i], 8 * kTqKt);
      mbar_init(&e_free[i], 1);
    }
    mbar_init(acc_final, 1);
    fence_barrier_init();
  }
  if (threadIdx.x >= 64 && threadIdx.x < 64 + kTqRows) {
    const int t = threadIdx.x - 64;
    const int hj = t / p.bt;
    const size_t ri = (size_t)min(row0 + t - hj * p.bt, p.R - 1) * p.Hq + min(h + hj, p.Hq - 1);
    rowp[t] = make_float2(p.lse[ri] * kLog2eTq, p.delta[ri]);
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
  const uint32_t tmem_st = tmem_base;           // two buffers of S^T [0,64) | T^T [64,128) of this CTA's 128 keys
  const uint32_t tmem_acc = tmem_base + 256;    // 3 x 64 columns: this CTA's 128 channels of each block

  if (warp == 0 || warp == 3) {
    // =========================================================== producers (two threads per CTA)
    // Two rings, one producer thread each (a single thread issues a TMA instruction every ~200
    // cycles, too slow for both): slots [0, kTqStSlots) carry K-major slabs (this CTA's 128 keys x
    // one channel group, two 64-token boxes) for [S^T | T^T], filled by warp 0; the rest carry
    // MN-major slots (64 keys of either CTA's tile x two of THIS CTA's channel groups, one box) for
    // dQ^T, filled by warp 3.  Every load credits the even CTA's barrier of the slot.
    if (lane == 0 && total_steps > 0) {
      const bool st_role = warp == 0;
      if (st_role) {
        if (leader) mbar_arrive_expect_tx(a_full, p.qdo_bytes);
        if (leader) {
          for (int c = 0; c < 8; ++c) tma_load_5d_pair(bop + c * 8192, &p.q_map, a_full, 0, row0, c, h, 0);
          tma_load_5d_pair(bop + kTqRope, &p.q_map, a_full, 0, row0, 8, h, 0);
        } else {
          for (int c = 0; c < 8; ++c) tma_load_5d_pair(bop + c * 8192, &p.do_map, a_full, 0, row0, c, h, 0);
          tma_load_5d_pair(bop + kTqRope - 4096, &p.q_map, a_full, 0, row0, 8, h, 0);
        }
      }
      const int pg_mask = (1 << p.pg_shift) - 1;
      bool ok = true;
      // a walk over the 256-key steps of the parts; a step is four 64-token boxes, resolved by `box`
      int part = part_lo, step = -1;
      int c_off = p.shard_page_offset[part], c_pages = p.shard_page_offset[part + 1] - c_off;
      int c_tail = p.shard_tail_slot[part], c_steps = (int)((((p.shard_tokens[part] + 127) >> 7) + 1) >> 1);
      auto next_step = [&]() {
        ++step;
        while (step >= c_steps) {          // (the caller stops after total_steps steps)
          ++part;
          step = 0;
          c_off = p.shard_page_offset[part];
          c_pages = p.shard_page_offset[part + 1] - c_off;
          c_tail = p.shard_tail_slot[part];
          c_steps = (int)((((p.shard_tokens[part] + 127) >> 7) + 1) >> 1);
        }
      };
      // box q of the step: physical page, first token inside it, and whether it is the pool's partly
      // filled last page.  Past the part's last page: a coordinate beyond the pool, where TMA fills zeros
      // (the bytes of an arbitrary page could be NaN patterns, and 0 * NaN would poison dQ^T).
      auto box = [&](int q, int& page, int& tok, bool& tail) {
        const int t = step * 256 + q * 64;
        const int ps = t >> p.pg_shift;
        page = ps < c_pages ? __ldg(p.shard_phys_pages + c_off + ps) : p.num_phys_pages;
        tok = t & pg_mask;
        tail = ps == c_tail;
      };
      uint32_t seq = 0, issued = 0;
      if (st_role) {
        for (int i = 0; i < total_steps && ok; ++i) {
          next_step();
          int pg0, pg1, tk0, tk1;
          bool tl0, tl1;
          box(2 * (int)rank, pg0, tk0, tl0);
          box(2 * (int)rank + 1, pg1, tk1, tl1);
          const CUtensorMap* m0 = tl0 ? &p.k_tail : &p.k_map;
          const CUtensorMap* m1 = tl1 ? &p.k_tail : &p.k_map;
#pragma unroll 1
          for (int c = 0; c < 9; ++c) {          // channel group c of this CTA's tile of the step
            const uint32_t slot = seq % kTqStSlots, lap = seq / kTqStSlots;
            ok = ok && LS_TQWAIT(tw0, mbar_wait(&empty[slot], (lap & 1) ^ 1, abort_flag));
            if (!ok) break;
            uint8_t* dst = ring + slot * kTqSlab;
            if (leader) mbar_arrive_expect_tx(&full[slot], 2 * kTqSlab);
            tma_load_5d_pair(dst, m0, &full[slot], 0, tk0, c, kvh, pg0);
            tma_load_5d_pair(dst + 8192, m1, &full[slot], 0, tk1, c, kvh, pg1);
            ++issued;
            ++seq;
          }
        }
        LS_TQDUMP(0, tw0);
        LS_TQDUMP(1, clock64() - t_begin);
      } else {
        const uint32_t full_remote = mapa_u32(smem_u32(&full[kTqStSlots]), 0);
        for (int i = 0; i < total_steps && ok; ++i) {
          next_step();
          int pg[4], tk[4];
          bool tl[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) box(q, pg[q], tk[q], tl[q]);
          // k = (tile of the step) * 6 + (channel block) * 2 + (64-key half): channel block m is groups
          // 4m, 4m+1 in the even CTA (group 9 does not exist and reads as zeros) and 4m+2, 4m+3 in the
          // odd CTA, which has nothing to load for block 2.
#pragma unroll
          for (int k = 0; k < 12; ++k) {
            const int j = k / 6, m = (k % 6) >> 1, q = 2 * j + (k & 1);
            const uint32_t sl = seq % kTqAccSlots, lap = seq / kTqAccSlots;
            const uint32_t slot = kTqStSlots + sl;
            ok = ok && LS_TQWAIT(tw1, mbar_wait(&empty[slot], (lap & 1) ^ 1, abort_flag));
            if (!ok) break;
            if (leader) mbar_arrive_expect_tx(&full[slot], m < 2 ? 2 * kTqSlab : kTqSlab / 2);
            else mbar_arrive_cluster(full_remote + sl * 8);
            if (m < 2)
              tma_load_5d_pair(ring + slot * kTqSlab, tl[q] ? &p.k2_tail : &p.k2_map, &full[slot], 0, tk[q],
                               4 * m + 2 * (int)rank, kvh, pg[q]);
            else if (leader)      // the rope group alone: the other half of the slot feeds accumulator lanes nobody reads
              tma_load_5d_pair(ring + slot * kTqSlab, tl[q] ? &p.k_tail : &p.k_map, &full[slot], 0, tk[q], 8, kvh,
                               pg[q]);
            ++issued;
            ++seq;
          }
        }
        LS_TQDUMP(2, tw1);
        LS_TQDUMP(3, clock64() - t_begin);
      }
      if (*abort_flag && leader) {   // aborted: wait (bounded) for the copies credited to this CTA's barriers
        const uint32_t per = st_role ? kTqStSlots : kTqAccSlots, first = st_role ? 0 : kTqStSlots;
        for (uint32_t idx = 0; idx < per && idx < issued; ++idx) {
          const uint32_t last_lap = (issued - 1 - idx) / per;
          const uint64_t t_start = globaltimer_ns();
          while (!mbar_try_wait(&full[first + idx], last_lap & 1, 1000) && globaltimer_ns() - t_start < 100000000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // =========================================================== [S^T | T^T] issuer (one thread of the even CTA)
    // The two kinds of products are issued by two threads (this one and one of warp 6), each
    // from its own ring: they write disjoint TMEM columns and each thread's own instructions
    // stay in order, so the per-slot bookkeeping of one overlaps the other's.
    if (leader && lane == 0 && total_steps > 0) {
      constexpr uint32_t idesc_st = make_idesc(256, 128, 0, 0);
      constexpr uint32_t idesc_rope = make_idesc(256, 64, 0, 0);
      constexpr uint32_t hi = sdesc_hi(1024);
      const uint32_t b_lo = sdesc_lo(smem_u32(bop), 16);
      const uint32_t ring_k_lo = sdesc_lo(smem_u32(ring), 16);          // K-major: 128 keys x 64 channels
      bool ok = mbar_wait(a_full, 0, abort_flag);
      uint32_t seq = 0;
      for (int i = 0; i < total_steps && ok; ++i) {
        if (i > 1) {      // the buffer's previous tile (step i - 2) is in registers
          ok = LS_TQWAIT(tw2, mbar_wait(&s_read[i & 1], ((i >> 1) - 1) & 1, abort_flag));
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
            mma_ss_pair(tmem_st + (i & 1) * 128, sdesc(a_lo + ((k * 32) >> 4), hi),
                        sdesc(b_lo + (((c < 8 ? c * 8192 : kTqRope) + k * 32) >> 4), hi),
                        c < 8 ? idesc_st : idesc_rope, (c | k) != 0);
          mma_commit_pair(&empty[slot]);
          ++seq;
        }
        if (!ok) break;
        mma_commit_pair(&st_full[i & 1]);
      }
      LS_TQDUMP(8, tw0);
      LS_TQDUMP(10, tw2);
      LS_TQDUMP(12, clock64() - t_begin);
    }
  } else if (warp == 2) {
    // =========================================================== dQ^T issuer (one thread of the even CTA)
    if (leader && lane == 0 && total_steps > 0) {
      constexpr uint32_t idesc_acc = make_idesc(256, 64, 1, 1);
      constexpr uint32_t hi = sdesc_hi(1024);
      constexpr uint32_t hi_e = sdesc_hi_sw64(512);
      const uint32_t ring_m_lo = sdesc_lo(smem_u32(ring), 8192);        // MN-major: 64 keys x two channel groups
      const uint32_t e_lo = sdesc_lo(smem_u32(e_smem), 512);            // MN-major, 64-byte lines: 128 keys x 32 rows per tile
      bool ok = true;
      uint32_t seq = 0;
      for (int i = 0; i < total_steps && ok; ++i) {
        ok = LS_TQWAIT(tw3, mbar_wait_cluster(&e_full[i & 1], (i >> 1) & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < 12; ++k) {
          const int j = k / 6, m = (k % 6) >> 1, kh = k & 1;
          const uint32_t slot = kTqStSlots + seq % kTqAccSlots, lap = seq / kTqAccSlots;
          ok = ok && LS_TQWAIT(tw1, mbar_wait(&full[slot], lap & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_lo = ring_m_lo + slot * (kTqSlab >> 4);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            mma_ss_pair(tmem_acc + m * 64, sdesc(a_lo + ((kk * 2048) >> 4), hi),
                        sdesc(e_lo + (((i & 1) * kTqE + j * 8192 + kh * 4096 + kk * 1024) >> 4), hi_e), idesc_acc,
                        (i | j | kh | kk) != 0);
          mma_commit_pair(&empty[slot]);
          ++seq;
        }
        if (!ok) break;
        mma_commit_pair(&e_free[i & 1]);
        if (i == total_steps - 1) mma_commit_pair(acc_final);
      }
      LS_TQDUMP(9, tw1);
      LS_TQDUMP(11, tw3);
      LS_TQDUMP(13, clock64() - t_begin);
    }
  } else {
    // =========================================================== two threads per key: E^T, epilogue
    // (thread `sub` of a key owns rows 32 sub .. 32 sub + 31, i.e. the half of E^T that lives in CTA `sub`;
    // with one thread per key -- one warp per scheduler -- these warps were busy 83 % of a step on TMEM-load,
    // MUFU and store latency that nothing overlapped)
    const int quad = warp & 3;
    const int sub = (warp - 4) >> 2;
    const int key = quad * 32 + lane;                      // TMEM lane = key of this CTA's tile
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    // E^T of this CTA's keys, MN-major [key][row] in 64-byte lines (64-byte swizzle): rows 0-31 go
    // to the even CTA's copy, rows 32-63 to the odd CTA's, each at offset rank * 8 KB of the E^T area
    const uint32_t e_mine = smem_u32(e_smem) + rank * 8192 + (key >> 3) * 512 + (key & 7) * 64;
    const uint32_t e_dst = mapa_u32(e_mine, (uint32_t)sub);
    const uint32_t sw = (uint32_t)(key & 7) >> 1;
    const uint32_t s_read_remote[2] = {mapa_u32(smem_u32(&s_read[0]), 0), mapa_u32(smem_u32(&s_read[1]), 0)};
    const uint32_t e_full_remote[2] = {mapa_u32(smem_u32(&e_full[0]), 0), mapa_u32(smem_u32(&e_full[1]), 0)};
    bool key_ok = true;
    if (total_steps > 0) {
      bool ok = true;
      int part = part_lo, step = -1;
      for (int i = 0; i < total_steps && ok; ++i) {
        ++step;
        while (step >= (int)((((p.shard_tokens[part] + 127) >> 7) + 1) >> 1)) {
          ++part;
          step = 0;
        }
        const bool valid = ((int64_t)(2 * step + (int)rank)) * 128 + key < p.shard_tokens[part];
        ok = LS_TQWAIT(tw0, mbar_wait(&st_full[i & 1], (i >> 1) & 1, abort_flag));
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tst = tmem_st + (i & 1) * 128 + lane_sel;
        uint32_t pk[16];
        {
          uint32_t sr[32], tr[32];
          tmem_ld32(tst + sub * 32, sr);
          tmem_ld32(tst + 64 + sub * 32, tr);
          tc_wait_ld32(sr);
          tc_wait_ld32(tr);
          tc_fence_before();        // this warp's share of the buffer is in registers: the next step may overwrite it
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(s_read_remote[i & 1]);
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            const float4 rp = *reinterpret_cast<const float4*>(rowp + sub * 32 + j);   // two rows
            const float p0 = ex2(fmaf(__uint_as_float(sr[j]), p.scale_log2, -rp.x));
            const float p1 = ex2(fmaf(__uint_as_float(sr[j + 1]), p.scale_log2, -rp.z));
            pk[j >> 1] = pack_bf16(p0 * (__uint_as_float(tr[j]) - rp.y), p1 * (__uint_as_float(tr[j + 1]) - rp.w));
          }
        }
        if (!valid) {
#pragma unroll
          for (int j = 0; j < 16; ++j) pk[j] = 0u;
        }
        if (i > 1) {      // the dQ^T instructions of step i - 2 have read this E^T buffer
          ok = LS_TQWAIT(tw1, mbar_wait(&e_free[i & 1], ((i >> 1) - 1) & 1, abort_flag));
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)          // 16-byte chunk: rows 32 sub + 8 q .. + 7, in CTA `sub`
          st_shared_cluster_v4(e_dst + (i & 1) * kTqE + (((uint32_t)q ^ sw) << 4), pk[4 * q], pk[4 * q + 1], pk[4 * q + 2],
                               pk[4 * q + 3]);
        fence_proxy_async_all();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster_release(e_full_remote[i & 1]);
      }
      if (threadIdx.x == 128) {
        LS_TQDUMP(16, tw0);
        LS_TQDUMP(17, tw1);
        LS_TQDUMP(18, clock64() - t_begin);
      }
      if (ok) ok = mbar_wait(acc_final, 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) tc_fence_after();
      key_ok = ok;
    }
    // ---- epilogue: this CTA's channels of the 64 rows.  Alone (one range of parts): scale, add the response
    // block's partial, write bf16.  Split: the fp32 sum goes to the range's scratch partial.  Chained: it is
    // added to the running dQ once the previous range's pair has published, and the last range writes bf16.
    const bool have_acc = total_steps > 0;
    const bool last = p.chain && split == p.nsplit - 1;
    const bool fold = p.chain && (split > 0 || p.acc_init);
    int* counter = p.chain ? p.ctl + kChainHeaderInts + kvh * p.nq_tiles + qtile : nullptr;
    if (key_ok && p.chain && split > 0)
      key_ok = __all_sync(0xffffffffu, chain_wait(counter, 2 * split, p.ctl, abort_flag));
    if (key_ok && (have_acc || p.nsplit > 1)) {
      const uint64_t pol = l2_policy_evict_first();     // the running dQ passes through L2 once per range
#pragma unroll 1
      for (int m = 0; m < 3; ++m) {
        if (m == 2 && (!leader || quad >= 2)) break;      // block 2 is the 64 rope channels, in the even CTA
        const int ch = m * 256 + (int)rank * 128 + key;
        {
          const int half = sub;             // this thread's 32 of the 64 rows
          uint32_t o[32];
          if (have_acc) {
            tmem_ld32(tmem_acc + lane_sel + m * 64 + half * 32, o);
            tc_wait_ld32(o);
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = 0u;
          }
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
              float v = __uint_as_float(o[j]);
              if (p.chain) {
                if (fold) v += ld_cg_hint_f32(p.dq_acc + idx, pol);
                if (last) p.dq[idx] = __float2bfloat16_rn(v * p.scale);
                else st_hint_f32(p.dq_acc + idx, v, pol);
              } else if (p.nsplit > 1) {
                p.dq_split[(size_t)split * p.R * p.Hq * 576 + idx] = v;
              } else {
                p.dq[idx] = __float2bfloat16_rn((v + (p.dq_resp ? p.dq_resp[idx] : 0.f)) * p.scale);
              }
            }
          }
        }
      }
    }
    if (p.chain) {
      const bool all_ok = bar_and(1, 128 * kTqKt, key_ok);      // every row of this CTA's channels is written
      if (key == 0 && sub == 0 && all_ok) chain_publish_add(counter);
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
    if (p.chain) st_relaxed_gpu(p.ctl + 1, 1);    // ends every other chain wait of this launch
  }
}

bool mla_dq_fast(const ls_pages* h) {
  const ls_pages_desc_t& d = h->desc;
  return d.dim_k == 576 && d.dim_v == 512 && d.v_aliases_k && d.prefix_len > 0;
}

int64_t mla_dq_blocks(const ls_pages* h, int R, int Hq) {
  const int Hkv = h->desc.num_kv_heads;
  return (int64_t)Hkv * row_tiling(R, Hq / Hkv, kTqRows).nq_tiles;
}

MlaDqSplit mla_dq_split(const ls_pages* h, int R, int Hq) {
  const int Hkv = h->desc.num_kv_heads;
  const int64_t blocks = (int64_t)Hkv * row_tiling(R, Hq / Hkv, kTqRows).nq_tiles;
  const int parts = h->prefix_parts();
  MlaDqSplit sp;
  if (blocks >= 74) {
    // a row block for every CTA pair of the GPU and more: ranges of whole parts holding up to 1.5 stream
    // budgets of keys (48 MB by default), the pairs of a range run together, so that its keys stay in L2
    // while every row block passes over them.  (Measured at the 1M workload, dQ pass: 19 MB ranges 325 ms,
    // 38 MB 314 ms, 75 MB 316 ms: shorter ranges pay the pair's prologue and hand-over more often, longer
    // ones start to fall out of L2.)
    const int64_t budget = ((h->desc.stream_budget_kib > 0 ? (int64_t)h->desc.stream_budget_kib : 32768ll) << 10) * 3 / 2;
    const int64_t part_bytes = std::max<int64_t>(1, h->desc.prefix_len * 576 * 2 / std::max(parts, 1));
    const int per_range = (int)std::max<int64_t>(1, std::min<int64_t>(parts, budget / part_bytes));
    sp.count = (parts + per_range - 1) / per_range;
    sp.chain = sp.count > 1;
  } else {
    // few rows: the parts are spread over enough CTA pairs to fill the GPU twice, all running at once
    sp.count = std::max(1, std::min(parts, (int)((148 + blocks - 1) / blocks)));
    sp.chain = false;
  }
  return sp;
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
                       const float* lse, const float* delta, float* dq_resp, float* scratch, int* ctl, void* dq,
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
  P.qdo_bytes = (9 + 9) * rt.bt * rt.bh * 128;      // Q (even CTA), dO and the rope slab of Q (odd CTA)
  MlaDqSplit sp = mla_dq_split(h, R, Hq);
  if (!scratch || !ctl) sp = MlaDqSplit{1, false};         // without scratch every pair walks all parts
  P.nsplit = sp.count;
  P.dq_split = scratch;
  P.chain = sp.chain ? 1 : 0;
  P.ctl = ctl;
  P.num_kv_heads = d.num_kv_heads;
  // chained: the running dQ starts as the response block's partial where there is one
  P.acc_init = dq_resp ? 1 : 0;
  P.dq_acc = dq_resp ? dq_resp : scratch;
  if (P.chain &&
      cudaMemsetAsync(ctl, 0, (kChainHeaderInts + (size_t)d.num_kv_heads * rt.nq_tiles) * sizeof(int), cs) != cudaSuccess)
    return LS_ERR_CUDA;
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
  const int64_t grid = (int64_t)d.num_kv_heads * rt.nq_tiles * P.nsplit * 2;     // CTA pairs
  if (grid > INT32_MAX) return LS_ERR_UNSUPPORTED_SHAPE;
  profile_begin(LS_KERNEL_BWD_DQ, cs);
  bwd_mla_dq_kernel<<<(int)grid, kTqThreads, kTqSmem, cs>>>(P);
  if (P.nsplit > 1 && !P.chain) {
    const int64_t n4 = (int64_t)R * Hq * 576 / 4;
    mla_dq_split_reduce_kernel<<<(int)std::min<int64_t>((n4 + 255) / 256, 148 * 8), 256, 0, cs>>>(
        scratch, P.nsplit, dq_resp, n4, prm->scale, static_cast<__nv_bfloat16*>(dq));
  }
  profile_end(LS_KERNEL_BWD_DQ, cs);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

}  // namespace ls
