// Folding the per-span pieces of the split attention into the block's attention output.
//
// Both tensor-core attention kernels cut a row's keys into aligned spans of SPAN_KEYS and leave, per (row, head, span),
// the span's score maximum (log2 domain), its sum of exponentials and its unnormalised output.  A (row, head) pair is
// folded by one warp: first the largest span maximum, then one weighted sum over the spans in ascending order.  The
// arithmetic involves the pair's own spans only, so it does not matter which kernel, CTA or warp runs it; it runs in
// the kernel that consumes the attention output (the output projection), spread over all its CTAs.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace fold {

constexpr int SPAN_KEYS = 512;

struct Params {
  const float *part;               // [rows][H][cap][HD + 2]; NULL: nothing to fold
  __nv_bfloat16 *out;              // [rows][H * HD]
  const int32_t *lin_end, *seg_len;   // per block row: keys seen = lin_end + seg_len
  const int *rows_dev;             // NULL, or the block's true row count in device memory
  int rows, H, cap, head_dim;
};

// Pairs first, first + step, .. (pair = row * H + head), two per pass so that their loads overlap.  Lane c fetches span
// c's maximum and sum (cap <= 32), then every lane fetches its dims of every span before the first is used.
template <int HD>
__device__ __forceinline__ void pairs(const Params &p, int rows, int first, int step, int lane) {
  constexpr int PW = HD + 2, DPL = HD / 32, UNR = 12;
  const int n_pairs = rows * p.H;
  for (int q0 = first; q0 < n_pairs; q0 += 2 * step) {
    const float *src[2];
    int ns[2];
    float m_l[2], l_l[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int q = q0 + k * step;
      ns[k] = 0;
      src[k] = p.part;
      if (q < n_pairs) {
        const int r = q / p.H;
        ns[k] = (p.lin_end[r] + p.seg_len[r] + SPAN_KEYS - 1) / SPAN_KEYS;
        src[k] = p.part + (size_t)q * p.cap * PW;
      }
      m_l[k] = -INFINITY;
      l_l[k] = 0.f;
      if (lane < ns[k]) {
        m_l[k] = __ldcg(src[k] + (size_t)lane * PW);
        l_l[k] = __ldcg(src[k] + (size_t)lane * PW + 1);
      }
    }
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      if (ns[k] == 0) continue;                                    // uniform in the warp
      float mx = m_l[k];
#pragma unroll
      for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float w_l = (m_l[k] == -INFINITY) ? 0.f : exp2f(m_l[k] - mx);   // mx is finite: the first span holds a visible key
      float l = 0.f, acc[DPL];
#pragma unroll
      for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
      for (int c0 = 0; c0 < ns[k]; c0 += UNR) {
        float o[UNR][DPL];
#pragma unroll
        for (int cc = 0; cc < UNR; ++cc)
#pragma unroll
          for (int i = 0; i < DPL; ++i)
            o[cc][i] = c0 + cc < ns[k] ? __ldcg(src[k] + (size_t)(c0 + cc) * PW + 2 + lane + 32 * i) : 0.f;
#pragma unroll
        for (int cc = 0; cc < UNR; ++cc) {
          if (c0 + cc >= ns[k]) break;                              // uniform in the warp
          const float w = __shfl_sync(0xffffffffu, w_l, c0 + cc);
          l += __shfl_sync(0xffffffffu, l_l[k], c0 + cc) * w;
#pragma unroll
          for (int i = 0; i < DPL; ++i) acc[i] += o[cc][i] * w;
        }
      }
      const float inv = 1.0f / l;
      __nv_bfloat16 *dst = p.out + (size_t)(q0 + k * step) * HD;
#pragma unroll
      for (int i = 0; i < DPL; ++i) dst[lane + 32 * i] = __float2bfloat16_rn(acc[i] * inv);
    }
  }
}

__device__ __forceinline__ void run(const Params &p, int first, int step, int lane) {
  const int rows = p.rows_dev ? min(p.rows, __ldg(p.rows_dev)) : p.rows;
  if (p.head_dim == 128) pairs<128>(p, rows, first, step, lane);
  else pairs<64>(p, rows, first, step, lane);
}

}  // namespace fold
