// Stable LSE/output merge of per-shard partials (Eq. qwen-lse-parts, Eq. qwen-global-attn):
//   m = max_r l_r;  a = sum_r e^{l_r - m};  n = sum_r e^{l_r - m} o_r;  o = n / a;  l = m + log a.
// HBM-bound: one warp per row, 16-byte vector loads, fp32 throughout -- or, BF16N, with the numerator
// carried the way the paper's production run exchanges it (Sec. "Global Full-Attention Forward
// Composition", last paragraph): every shard's term e^{l_r - m} o_r rounded to bf16 and the terms added in
// shard order with a bf16 running sum; maximum, denominator and l stay fp32.
#include <cuda_bf16.h>

#include "ls_internal.h"

namespace ls {

constexpr int kMergeWarps = 8;

__device__ __forceinline__ float bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

template <bool BF16N>
__global__ void __launch_bounds__(kMergeWarps * 32) merge_kernel(int num_parts, int64_t rows, int dv,
                                                                 const float* __restrict__ o_part,
                                                                 const float* __restrict__ lse_part,
                                                                 __nv_bfloat16* __restrict__ o_bf16,
                                                                 float* __restrict__ o_f32,
                                                                 float* __restrict__ lse_out,
                                                                 int32_t* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * kMergeWarps + (threadIdx.x >> 5);
  if (row >= rows) return;
  float m = -INFINITY;
  for (int r = lane; r < num_parts; r += 32) m = fmaxf(m, lse_part[(int64_t)r * rows + row]);
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  const float m_safe = (m == -INFINITY) ? 0.f : m;
  float a = 0.f;
  for (int r = lane; r < num_parts; r += 32) a += expf(lse_part[(int64_t)r * rows + row] - m_safe);
  for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
  const float inv_a = a > 0.f ? 1.f / a : 0.f;
  for (int c = lane * 4; c < dv; c += 128) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int r = 0; r < num_parts; ++r) {
      const float w = expf(lse_part[(int64_t)r * rows + row] - m_safe);
      if (w == 0.f) continue;     // an empty partial weighs exactly nothing
      const float4 v = *reinterpret_cast<const float4*>(o_part + ((int64_t)r * rows + row) * dv + c);
      if (BF16N) {
        acc.x = bf16_round(acc.x + bf16_round(w * v.x));
        acc.y = bf16_round(acc.y + bf16_round(w * v.y));
        acc.z = bf16_round(acc.z + bf16_round(w * v.z));
        acc.w = bf16_round(acc.w + bf16_round(w * v.w));
      } else {
        acc.x = fmaf(w, v.x, acc.x);
        acc.y = fmaf(w, v.y, acc.y);
        acc.z = fmaf(w, v.z, acc.z);
        acc.w = fmaf(w, v.w, acc.w);
      }
    }
    acc.x *= inv_a;
    acc.y *= inv_a;
    acc.z *= inv_a;
    acc.w *= inv_a;
    if (o_f32) *reinterpret_cast<float4*>(o_f32 + row * dv + c) = acc;
    if (o_bf16) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&lo);
      pk.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(o_bf16 + row * dv + c) = pk;
    }
  }
  if (lane == 0) {
    // a = 0 with m = -inf is the all-empty row (l = -inf); NaN or +inf can only come from non-finite inputs
    const float l = (a > 0.f || a != a) ? m_safe + logf(a) : -INFINITY;
    lse_out[row] = l;
    if (status && (l != l || l == INFINITY)) atomicExch(status, (int)LS_ERR_NONFINITE);
  }
}

}  // namespace ls

static ls_status_t launch_merge(bool bf16n, int32_t num_parts, int64_t rows, int32_t dim_v, const float* o_part,
                                const float* lse_part, void* o_bf16, float* o_f32, float* lse, int32_t* status_dev,
                                void* stream) {
  if (num_parts < 1 || rows < 0 || dim_v < 4 || dim_v % 4 != 0) return LS_ERR_INVALID_ARG;
  if (!o_part || !lse_part || !lse) return LS_ERR_INVALID_ARG;
  if (!ls::aligned16(o_part) || (o_f32 && !ls::aligned16(o_f32)) || (o_bf16 && !ls::aligned16(o_bf16)))
    return LS_ERR_ALIGNMENT;
  if (rows == 0) return LS_OK;
  const int64_t blocks = (rows + ls::kMergeWarps - 1) / ls::kMergeWarps;
  if (blocks > INT32_MAX) return LS_ERR_UNSUPPORTED_SHAPE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (bf16n)
    ls::merge_kernel<true><<<(int)blocks, ls::kMergeWarps * 32, 0, cs>>>(
        num_parts, rows, dim_v, o_part, lse_part, static_cast<__nv_bfloat16*>(o_bf16), o_f32, lse, status_dev);
  else
    ls::merge_kernel<false><<<(int)blocks, ls::kMergeWarps * 32, 0, cs>>>(
        num_parts, rows, dim_v, o_part, lse_part, static_cast<__nv_bfloat16*>(o_bf16), o_f32, lse, status_dev);
  return cudaGetLastError() == cudaSuccess ? LS_OK : LS_ERR_CUDA;
}

extern "C" ls_status_t ls_lse_merge(int32_t num_parts, int64_t rows, int32_t dim_v, const float* o_part,
                                    const float* lse_part, void* o_bf16, float* o_f32, float* lse,
                                    int32_t* status_dev, void* stream) {
  return launch_merge(false, num_parts, rows, dim_v, o_part, lse_part, o_bf16, o_f32, lse, status_dev, stream);
}

extern "C" ls_status_t ls_lse_merge_bf16_numerator(int32_t num_parts, int64_t rows, int32_t dim_v, const float* o_part,
                                                   const float* lse_part, void* o_bf16, float* o_f32, float* lse,
                                                   int32_t* status_dev, void* stream) {
  return launch_merge(true, num_parts, rows, dim_v, o_part, lse_part, o_bf16, o_f32, lse, status_dev, stream);
}
