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
// TMEM columns: O [0, DV), S/P buffer 0 [DV, DV+128), S/P buffer 1 [DV+128, DV+256).
// K chunk  = 128 keys x 64 channels (K-major, 128-byte swizzle): one k-slice of S.
// V chunk  = VKEYS keys x DV channels as DV/64 sub-slabs (MN-major): VKEYS/16 k-steps of PV.
#include "ls_internal.h"
#include "ls_sm100.cuh"

namespace ls {

struct FwdParams {
  CUtensorMap q_map;
  CUtensorMap k_map, k_tail_map;
  CUtensorMap v_map, v_tail_map;
  CUtensorMap kr_map, vr_map;
  const int32_t* shard_phys_pages;
  const int32_t* shard_page_offset;
  const int32_t* shard_tail_slot;
  const int64_t* shard_tokens;
  float* o_part;
  float* lse_part;
  int32_t* status;
  int R, Hq, Hkv, g, S, pg, box_tok_k, tiles_per_head, nq_tiles, num_phys_pages;
  float scale, scale_log2;
};

constexpr int kChunkBytes = 16384;
constexpr int kFwdThreads = 192;
constexpr float kRescaleLog2 = 8.0f;   // the reference max lags the true max by at most 2^8

template <int DK, int DV>
struct FwdCfg {
  static constexpr int KCH = DK / 64;            // K chunks per 128-key tile
  static constexpr int VKEYS = 8192 / DV;        // keys per V chunk
  static constexpr int NVCH = 128 / VKEYS;       // V chunks per tile
  static constexpr int RING = (DK == 128) ? 10 : 8;
  static constexpr int Q_BYTES = KCH * kChunkBytes;
  static constexpr int SMEM_BYTES = 1024 + Q_BYTES + RING * kChunkBytes + 512;
};

template <int DK, int DV>
__global__ void __launch_bounds__(kFwdThreads, 1) fwd_kernel(const __grid_constant__ FwdParams p) {
  using C = FwdCfg<DK, DV>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_smem = smem;
  uint8_t* ring = smem + C::Q_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + C::RING * kChunkBytes);
  uint64_t* q_full = bars;
  uint64_t* full = bars + 1;
  uint64_t* empty = full + C::RING;
  uint64_t* s_full = empty + C::RING;   // [2]
  uint64_t* p_full = s_full + 2;        // [2]
  uint64_t* pv_done = p_full + 2;       // one phase per tile: O += P V of that tile finished
  uint64_t* o_final = pv_done + 1;      // the last tile's P V finished
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(o_final + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- work item
  int idx = blockIdx.x;
  const int qtile = idx % p.nq_tiles;
  idx /= p.nq_tiles;
  const int part = idx % (p.S + 1);
  const int kvh = idx / (p.S + 1);
  const int h = kvh * p.g + qtile / p.tiles_per_head;
  const int ttile = qtile % p.tiles_per_head;
  const int t0 = ttile * 128;
  const bool is_resp = (part == p.S);
  int64_t tokens;
  int page_off = 0, n_pages = 0, tail_slot = -1;
  if (is_resp) {
    tokens = min(p.R, t0 + 128);                       // keys 0 .. last row of this tile
  } else {
    tokens = p.shard_tokens[part];
    page_off = p.shard_page_offset[part];
    n_pages = p.shard_page_offset[part + 1] - page_off;
    tail_slot = p.shard_tail_slot[part];
  }
  const int n_tiles = (int)((tokens + 127) / 128);

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

  if (warp == 0) {
    // =========================================================== producer
    if (n_tiles > 0) {
      if (lane == 0) {
        mbar_arrive_expect_tx(q_full, C::Q_BYTES);
        for (int c = 0; c < C::KCH; ++c) tma_load_4d(q_smem + c * kChunkBytes, &p.q_map, q_full, c * 64, t0, h, 0);
      }
      const int32_t* pages = p.shard_phys_pages + page_off;
      int win_tag[2] = {-1, -1};
      int win_page[2] = {0, 0};
      // physical page of the shard's page slot `ps` (warp-uniform); out of range -> a page
      // coordinate past the pool, which TMA fills with zeros
      auto page_of = [&](int ps) -> int {
        const int w = ps >> 5, b = w & 1;
        if (win_tag[b] != w) {
          win_tag[b] = w;
          const int i = (w << 5) + lane;
          win_page[b] = (i < n_pages) ? __ldg(pages + i) : p.num_phys_pages;
        }
        return __shfl_sync(0xffffffffu, win_page[b], ps & 31);
      };
      uint32_t cc = 0;      // chunks issued so far
      bool ok = true;
      auto acquire = [&]() -> uint8_t* {          // lane 0 only
        const uint32_t slot = cc % C::RING, ph = (cc / C::RING) & 1;
        ok = ok && mbar_wait(&empty[slot], ph ^ 1, abort_flag);
        if (ok) mbar_arrive_expect_tx(&full[slot], kChunkBytes);
        return ring + slot * kChunkBytes;
      };
      auto load_k = [&](int tile) {
        const int box_tok = is_resp ? 128 : p.box_tok_k;   // the response maps use 128-token boxes
        const int nbox = 128 / box_tok;
        int pg_id[2], off[2], tl[2];
        for (int b = 0; b < nbox; ++b) {
          const int tok = tile * 128 + b * box_tok;
          if (is_resp) { pg_id[b] = 0; off[b] = tok; tl[b] = 0; }
          else {
            const int ps = tok / p.pg;
            pg_id[b] = page_of(ps);
            off[b] = tok % p.pg;
            tl[b] = (ps == tail_slot);
          }
        }
        if (lane == 0) {
          for (int c = 0; c < C::KCH; ++c) {
            uint8_t* dst = acquire();
            if (ok) {
              for (int b = 0; b < nbox; ++b) {
                const CUtensorMap* m = is_resp ? &p.kr_map : (tl[b] ? &p.k_tail_map : &p.k_map);
                tma_load_4d(dst + b * box_tok * 128, m, &full[cc % C::RING], c * 64, off[b], kvh, pg_id[b]);
              }
            }
            ++cc;
          }
        }
      };
      auto load_v = [&](int tile) {
        int pg_id[C::NVCH], off[C::NVCH], tl[C::NVCH];
        for (int r = 0; r < C::NVCH; ++r) {
          const int tok = tile * 128 + r * C::VKEYS;
          if (is_resp) { pg_id[r] = 0; off[r] = tok; tl[r] = 0; }
          else {
            const int ps = tok / p.pg;
            pg_id[r] = page_of(ps);
            off[r] = tok % p.pg;
            tl[r] = (ps == tail_slot);
          }
        }
        if (lane == 0) {
          for (int r = 0; r < C::NVCH; ++r) {
            uint8_t* dst = acquire();
            if (ok) {
              const CUtensorMap* m = is_resp ? &p.vr_map : (tl[r] ? &p.v_tail_map : &p.v_map);
              for (int c = 0; c < DV / 64; ++c)
                tma_load_4d(dst + c * C::VKEYS * 128, m, &full[cc % C::RING], c * 64, off[r], kvh, pg_id[r]);
            }
            ++cc;
          }
        }
      };
      load_k(0);
      for (int i = 0; i < n_tiles; ++i) {
        if (i + 1 < n_tiles) load_k(i + 1);
        load_v(i);
      }
      // On an aborted run, wait (bounded) until every copy this thread started has landed.
      if (lane == 0 && *abort_flag) {
        for (uint32_t s = 0; s < (uint32_t)C::RING && s < cc; ++s) {
          const uint32_t last = ((cc - 1 - s) / C::RING) * C::RING + s;   // last chunk index in slot s
          const uint64_t t_start = globaltimer_ns();
          while (!mbar_try_wait(&full[s], (last / C::RING) & 1) && globaltimer_ns() - t_start < 100000000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // =========================================================== MMA issuer
    if (lane == 0 && n_tiles > 0) {
      constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);
      constexpr uint32_t idesc_pv = make_idesc(128, DV, 0, 1);
      const uint32_t q_addr = smem_u32(q_smem);
      const uint32_t ring_addr = smem_u32(ring);
      uint32_t cc = 0;
      bool ok = mbar_wait(q_full, 0, abort_flag);
      auto issue_s = [&](int tile) {
        const uint32_t d = tmem_s0 + (tile & 1) * 128;
        for (int c = 0; c < C::KCH; ++c) {
          const uint32_t slot = cc % C::RING, ph = (cc / C::RING) & 1;
          ok = ok && mbar_wait(&full[slot], ph, abort_flag);
          if (!ok) return;
          tc_fence_after();
          const uint32_t a0 = q_addr + c * kChunkBytes, b0 = ring_addr + slot * kChunkBytes;
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_ss(d, make_sdesc(a0 + k * 32, 16, 1024), make_sdesc(b0 + k * 32, 16, 1024), idesc_s,
                   (c | k) != 0);
          mma_commit(&empty[slot]);
          ++cc;
        }
        mma_commit(&s_full[tile & 1]);
      };
      auto issue_pv = [&](int tile) {
        const uint32_t a_base = tmem_s0 + (tile & 1) * 128;   // P over the S columns
        for (int r = 0; r < C::NVCH; ++r) {
          const uint32_t slot = cc % C::RING, ph = (cc / C::RING) & 1;
          ok = ok && mbar_wait(&full[slot], ph, abort_flag);
          if (!ok) return;
          tc_fence_after();
          const uint32_t b0 = ring_addr + slot * kChunkBytes;
#pragma unroll
          for (int kk = 0; kk < C::VKEYS / 16; ++kk)
            mma_ts(tmem_o, a_base + (r * (C::VKEYS / 16) + kk) * 8, make_sdesc(b0 + kk * 2048, C::VKEYS * 128, 1024),
                   idesc_pv, (tile | r | kk) != 0);
          mma_commit(&empty[slot]);
          ++cc;
        }
        mma_commit(pv_done);
        if (tile == n_tiles - 1) mma_commit(o_final);
      };
      if (ok) issue_s(0);
      for (int i = 0; i < n_tiles && ok; ++i) {
        if (i + 1 < n_tiles) issue_s(i + 1);
        ok = ok && mbar_wait(&p_full[i & 1], (i >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        issue_pv(i);
      }
    }
  } else {
    // =========================================================== softmax + epilogue
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int t = t0 + row;
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    const size_t out_row = ((size_t)part * p.R + (size_t)min(t, p.R - 1)) * p.Hq + h;
    float* o_dst = p.o_part + out_row * DV;
    if (n_tiles == 0) {
      if (t < p.R) {
        for (int c = 0; c < DV; c += 4) *reinterpret_cast<float4*>(o_dst + c) = make_float4(0.f, 0.f, 0.f, 0.f);
        p.lse_part[out_row] = -INFINITY;
      }
    } else {
      // last visible key index of this row inside this partial
      const int64_t lim = is_resp ? (int64_t)min(t, p.R - 1) : tokens - 1;
      float m_ref = -INFINITY, l = 0.f;
      const float thresh = kRescaleLog2 / p.scale_log2;
      bool ok = true;
      for (int i = 0; i < n_tiles && ok; ++i) {
        const uint32_t ts = tmem_s0 + (i & 1) * 128 + lane_sel;
        ok = mbar_wait(&s_full[i & 1], (i >> 1) & 1, abort_flag);
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
        } else if (__any_sync(0xffffffffu, mx > m_ref + thresh)) {
          // rare: raise the reference maximum and rescale the running sum and O
          ok = mbar_wait(pv_done, (i - 1) & 1, abort_flag);
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
      if (ok) ok = mbar_wait(o_final, 0, abort_flag);
      if (ok) {
        tc_fence_after();
        const float inv_l = (l > 0.f) ? 1.0f / l : 0.f;
#pragma unroll 1
        for (int c = 0; c < DV; c += 32) {
          uint32_t o[32];
          tmem_ld32(tmem_o + lane_sel + c, o);
          tc_wait_ld32(o);
          if (t < p.R) {
#pragma unroll
            for (int j = 0; j < 32; j += 4)
              *reinterpret_cast<float4*>(o_dst + c + j) =
                  make_float4(__uint_as_float(o[j]) * inv_l, __uint_as_float(o[j + 1]) * inv_l,
                              __uint_as_float(o[j + 2]) * inv_l, __uint_as_float(o[j + 3]) * inv_l);
          }
        }
        if (t < p.R) p.lse_part[out_row] = (l > 0.f) ? m_ref * p.scale + logf(l) : -INFINITY;
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

template <int DK, int DV>
static ls_status_t launch_fwd(const FwdParams& prm, int grid, cudaStream_t st) {
  using C = FwdCfg<DK, DV>;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(fwd_kernel<DK, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) !=
        cudaSuccess)
      return LS_ERR_CUDA;
    configured = true;
  }
  profile_begin(LS_KERNEL_FWD, st);
  fwd_kernel<DK, DV><<<grid, kFwdThreads, C::SMEM_BYTES, st>>>(prm);
  profile_end(LS_KERNEL_FWD, st);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

}  // namespace ls

extern "C" size_t ls_replay_attn_workspace_bytes(const ls_pages_t* h, const ls_attn_params_t* prm, int which) {
  if (!h || !prm || prm->R < 1 || prm->num_q_heads < 1) return 0;
  if (which == LS_WORKSPACE_FWD) return 0;
  // backward: per-partial dQ (fp32) + Delta (fp32)
  const size_t rows = (size_t)prm->R * prm->num_q_heads;
  return (size_t)(h->desc.num_shards + 1) * rows * h->desc.dim_k * sizeof(float) + rows * sizeof(float);
}

extern "C" ls_status_t ls_replay_attn_fwd(const ls_pages_t* h, const ls_attn_params_t* prm, const void* q,
                                          const void* k_resp, const void* v_resp, float* o_part, float* lse_part,
                                          void* workspace, size_t workspace_bytes, int32_t* status_dev,
                                          void* stream) {
  (void)workspace;
  (void)workspace_bytes;
  if (!h || !prm || !q || !k_resp || !v_resp || !o_part || !lse_part) return LS_ERR_INVALID_ARG;
  if (!h->on_device) return LS_ERR_INVALID_ARG;
  const ls_pages_desc_t& d = h->desc;
  if (prm->R < 1 || prm->num_q_heads < 1 || prm->num_q_heads % d.num_kv_heads != 0) return LS_ERR_INVALID_ARG;
  if (!(prm->scale > 0.f)) return LS_ERR_INVALID_ARG;
  if (!ls::aligned16(q) || !ls::aligned16(k_resp) || !ls::aligned16(v_resp) || !ls::aligned16(o_part))
    return LS_ERR_ALIGNMENT;
  if (!((d.dim_k == 128 && d.dim_v == 128) || (d.dim_k == 256 && d.dim_v == 256))) return LS_ERR_UNSUPPORTED_SHAPE;

  ls::FwdParams P;
  const int R = prm->R, Hq = prm->num_q_heads, Hkv = d.num_kv_heads;
  const int vkeys = 8192 / d.dim_v;
  const int box_k = d.page_size >= 128 ? 128 : 64;
  ls_status_t st = ls::encode_map(&P.q_map, q, d.dim_k, R, Hq, 1, (int64_t)Hq * d.dim_k, d.dim_k,
                                  (int64_t)R * Hq * d.dim_k, 128);
  if (st == LS_OK)
    st = ls::encode_map(&P.kr_map, k_resp, d.dim_k, R, Hkv, 1, (int64_t)Hkv * d.dim_k, d.dim_k,
                        (int64_t)R * Hkv * d.dim_k, 128);
  if (st == LS_OK)
    st = ls::encode_map(&P.vr_map, v_resp, d.dim_v, R, Hkv, 1, (int64_t)Hkv * d.dim_v, d.dim_v,
                        (int64_t)R * Hkv * d.dim_v, vkeys);
  if (st != LS_OK) return st;
  P.k_map = h->k_maps.full[ls::box_index(box_k)];
  P.k_tail_map = h->k_maps.tail[ls::box_index(box_k)];
  P.v_map = h->v_maps.full[ls::box_index(vkeys)];
  P.v_tail_map = h->v_maps.tail[ls::box_index(vkeys)];
  P.shard_phys_pages = h->d_shard_phys_pages;
  P.shard_page_offset = h->d_shard_page_offset;
  P.shard_tail_slot = h->d_shard_tail_slot;
  P.shard_tokens = h->d_shard_tokens;
  P.o_part = o_part;
  P.lse_part = lse_part;
  P.status = status_dev;
  P.R = R;
  P.Hq = Hq;
  P.Hkv = Hkv;
  P.g = Hq / Hkv;
  P.S = d.num_shards;
  P.pg = d.page_size;
  P.box_tok_k = box_k;
  P.tiles_per_head = (R + 127) / 128;
  P.nq_tiles = P.g * P.tiles_per_head;
  P.num_phys_pages = (int)std::min<int64_t>(d.num_phys_pages, INT32_MAX);
  P.scale = prm->scale;
  P.scale_log2 = prm->scale * 1.4426950408889634f;
  const int64_t grid = (int64_t)Hkv * (d.num_shards + 1) * P.nq_tiles;
  if (grid > INT32_MAX) return LS_ERR_UNSUPPORTED_SHAPE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (d.dim_k == 128) return ls::launch_fwd<128, 128>(P, (int)grid, cs);
  return ls::launch_fwd<256, 256>(P, (int)grid, cs);
}
