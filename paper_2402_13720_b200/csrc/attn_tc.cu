// Candidate-masked attention over the KV cache for a block of query rows (bf16, tensor cores, split along keys).
//
// Section 3.2 of the paper verifies K lengthened drafts in one forward by masking attention so that a phrase
// suffix sees the prefix, the draft and itself only (Eq. 8).  Here that mask is never materialised: a row is
// described by the number of keys it sees and by where its last keys live (its own candidate's cache slots),
// and the kernel maps "virtual positions" 0..n_vis-1 to cache slots on the fly.
//
// Work split.  Keys are cut by virtual position into aligned chunks of 256; one CTA handles one (kv head,
// chunk): it stages the chunk's K and V rows in shared memory once and serves every query row and every query
// head of the group from there, so each cached byte is read from HBM once.  Inside the CTA each of the 8 warps
// owns 32 keys, computes S = Q K^T, a local softmax and P V with mma.sync for 16 query rows at a time, and the 8
// warp results are folded in warp order into the chunk's (max, sum, output) triple.  A second kernel folds the
// chunks of a row in ascending order and normalises.
//
// Chunks below the cache length are the same for all rows.  The chunk(s) holding the block's own keys differ
// between the trunk and each candidate: the CTA keeps the shared part of the tile and swaps in each group's own
// rows in turn.  The value computed for a query depends only on (virtual position -> key) and on fixed chunk and
// warp boundaries, never on the other rows of the block, so a token gets bit-identical attention whether it is
// verified inside a candidate block or decoded alone.
#include "ouro_internal.h"

namespace {

constexpr int CH = 256;            // keys per chunk
constexpr int WARPS = 8;
constexpr int KW = CH / WARPS;     // keys per warp
constexpr int THREADS = WARPS * 32;

struct AttnParams {
  const __nv_bfloat16 *q;          // [rows][H*HD] rotated queries
  const __nv_bfloat16 *k, *v;      // this layer's cache: [max_seq][Hkv*HD]
  const int32_t *lin_end, *seg_start, *seg_len, *group;
  int rows, H, Hkv, L, cap;        // L: cache length before the block; cap: chunk slots per (row, head)
  float scale_log2;
  float *part;                     // [rows][H][cap][HD+2]: max (log2 domain), sum, unnormalised output
  __nv_bfloat16 *out;              // [rows][H*HD]
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float *d, const uint32_t *a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&t);
}
// log2-domain running softmax state folded with another piece: exact no-op when the piece is empty
__device__ __forceinline__ void fold_scales(float m, float mp, float &m_new, float &a, float &b) {
  m_new = fmaxf(m, mp);
  a = (m == -INFINITY) ? 0.f : exp2f(m - m_new);
  b = (mp == -INFINITY) ? 0.f : exp2f(mp - m_new);
}

template <int HD>
__global__ void __launch_bounds__(THREADS) attn_chunk_kernel(const AttnParams p) {
  constexpr int CPR = HD / 8;                 // 16-byte pieces per row
  constexpr int ROWB = HD * 2;                // bytes per tile row
  constexpr int PW = HD + 2;                  // floats per partial
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t *Ks = smem, *Vs = smem + CH * ROWB;
  float *mbuf = (float *)(smem + 2 * CH * ROWB);          // [WARPS][16][PW]
  int *s_nvis = (int *)(mbuf + WARPS * 16 * PW);          // [OURO_MAX_ROWS]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int c = blockIdx.x, kvh = blockIdx.y, c0 = c * CH;
  const int g = p.H / p.Hkv, dkv = p.Hkv * HD;
  const uint32_t ks_u = smem_u32(Ks), vs_u = smem_u32(Vs);
  const int key0 = warp * KW;                 // first tile row of this warp

  for (int r = threadIdx.x; r < p.rows; r += THREADS) s_nvis[r] = p.lin_end[r] + p.seg_len[r];

  // ---- stage the part of the chunk that every row shares (positions below the cache length); zero the rest
  for (int idx = lane; idx < KW * CPR; idx += 32) {
    int row = key0 + idx / CPR, ch = idx % CPR, pos = c0 + row;
    uint32_t off = row * ROWB + ((ch ^ (row & 7)) << 4);
    if (pos < p.L) {
      size_t src = (size_t)pos * dkv + kvh * HD + ch * 8;
      cp_async16(ks_u + off, p.k + src);
      cp_async16(vs_u + off, p.v + src);
    } else {
      *reinterpret_cast<uint4 *>(Ks + off) = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4 *>(Vs + off) = make_uint4(0, 0, 0, 0);
    }
  }
  cp_commit();
  __syncthreads();                            // s_nvis visible

  const bool common = c0 + CH <= p.L;
  int g_begin = 0;
  while (g_begin < p.rows) {
    // ---- one pass: all rows (shared chunk) or the rows of one group (chunk holding block keys)
    int g_end = p.rows, lin_g = INT_MAX, seg_g = 0;
    if (!common) {
      int gid = p.group[g_begin];
      g_end = g_begin + 1;
      while (g_end < p.rows && p.group[g_end] == gid) ++g_end;
      int last = g_end - 1;
      if (p.seg_len[last] > 0) { lin_g = p.lin_end[last]; seg_g = p.seg_start[last]; }
      int nv_max = s_nvis[last];
      if (nv_max > c0) {
        // this group's own keys: virtual positions [max(c0, L), min(c0 + CH, nv_max)) of the warp's 32 rows
        for (int idx = lane; idx < KW * CPR; idx += 32) {
          int row = key0 + idx / CPR, ch = idx % CPR, pos = c0 + row;
          if (pos >= p.L && pos < nv_max) {
            int slot = pos < lin_g ? pos : seg_g + (pos - lin_g);
            uint32_t off = row * ROWB + ((ch ^ (row & 7)) << 4);
            size_t src = (size_t)slot * dkv + kvh * HD + ch * 8;
            cp_async16(ks_u + off, p.k + src);
            cp_async16(vs_u + off, p.v + src);
          }
        }
        cp_commit();
      }
    }
    cp_wait_all();
    __syncwarp();

    const int nr = g_end - g_begin, M = g * nr;
    for (int mt = 0; mt * 16 < M; ++mt) {
      // the two query rows of this thread
      const int mA = mt * 16 + (lane >> 2), mB = mA + 8;
      const bool vA = mA < M, vB = mB < M;
      const int rA = g_begin + (vA ? mA % nr : 0), rB = g_begin + (vB ? mB % nr : 0);
      const int hA = kvh * g + (vA ? mA / nr : 0), hB = kvh * g + (vB ? mB / nr : 0);
      const int nvA = vA ? s_nvis[rA] : 0, nvB = vB ? s_nvis[rB] : 0;
      // skip tiles none of whose rows reaches this chunk (their partial is never read); same in every warp
      if (__ballot_sync(0xffffffffu, nvA > c0 || nvB > c0) == 0) continue;

      const __nv_bfloat16 *qA = p.q + (size_t)rA * p.H * HD + hA * HD + 2 * (lane & 3);
      const __nv_bfloat16 *qB = p.q + (size_t)rB * p.H * HD + hB * HD + 2 * (lane & 3);
      float s[4][4];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < HD / 16; ++ks) {
        uint32_t a[4];
        a[0] = vA ? *reinterpret_cast<const uint32_t *>(qA + 16 * ks) : 0u;
        a[1] = vB ? *reinterpret_cast<const uint32_t *>(qB + 16 * ks) : 0u;
        a[2] = vA ? *reinterpret_cast<const uint32_t *>(qA + 16 * ks + 8) : 0u;
        a[3] = vB ? *reinterpret_cast<const uint32_t *>(qB + 16 * ks + 8) : 0u;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          int mi = lane >> 3;
          int row = key0 + 16 * half + (lane & 7) + ((mi >> 1) << 3);
          int ch = 2 * ks + (mi & 1);
          uint32_t b0, b1, b2, b3;
          ldsm_x4(ks_u + row * ROWB + ((ch ^ (row & 7)) << 4), b0, b1, b2, b3);
          mma16816(s[2 * half], a, b0, b1);
          mma16816(s[2 * half + 1], a, b2, b3);
        }
      }
      // mask by virtual position, local softmax over this warp's 32 keys (log2 domain)
      float mxA = -INFINITY, mxB = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        int kp = c0 + key0 + 8 * nt + 2 * (lane & 3);
        s[nt][0] = kp < nvA ? s[nt][0] * p.scale_log2 : -INFINITY;
        s[nt][1] = kp + 1 < nvA ? s[nt][1] * p.scale_log2 : -INFINITY;
        s[nt][2] = kp < nvB ? s[nt][2] * p.scale_log2 : -INFINITY;
        s[nt][3] = kp + 1 < nvB ? s[nt][3] * p.scale_log2 : -INFINITY;
        mxA = fmaxf(mxA, fmaxf(s[nt][0], s[nt][1]));
        mxB = fmaxf(mxB, fmaxf(s[nt][2], s[nt][3]));
      }
      mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 1));
      mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 2));
      mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 1));
      mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 2));
      const float uA = mxA == -INFINITY ? 0.f : mxA, uB = mxB == -INFINITY ? 0.f : mxB;
      float lA = 0.f, lB = 0.f;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        s[nt][0] = exp2f(s[nt][0] - uA);
        s[nt][1] = exp2f(s[nt][1] - uA);
        s[nt][2] = exp2f(s[nt][2] - uB);
        s[nt][3] = exp2f(s[nt][3] - uB);
        lA += s[nt][0] + s[nt][1];
        lB += s[nt][2] + s[nt][3];
      }
      lA += __shfl_xor_sync(0xffffffffu, lA, 1);
      lA += __shfl_xor_sync(0xffffffffu, lA, 2);
      lB += __shfl_xor_sync(0xffffffffu, lB, 1);
      lB += __shfl_xor_sync(0xffffffffu, lB, 2);
      // O = P V over the warp's 32 keys
      float o[HD / 8][4];
#pragma unroll
      for (int nt = 0; nt < HD / 8; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
#pragma unroll
      for (int kk = 0; kk < 2; ++kk) {
        uint32_t a[4];
        a[0] = pack_bf16(s[2 * kk][0], s[2 * kk][1]);
        a[1] = pack_bf16(s[2 * kk][2], s[2 * kk][3]);
        a[2] = pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]);
        a[3] = pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
        for (int np = 0; np < HD / 16; ++np) {
          int mi = lane >> 3;
          int row = key0 + 16 * kk + (lane & 7) + ((mi & 1) << 3);
          int ch = 2 * np + (mi >> 1);
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(vs_u + row * ROWB + ((ch ^ (row & 7)) << 4), b0, b1, b2, b3);
          mma16816(o[2 * np], a, b0, b1);
          mma16816(o[2 * np + 1], a, b2, b3);
        }
      }
      // park the warp's piece, then fold the 8 pieces in warp order
      float *mineA = mbuf + ((size_t)warp * 16 + (lane >> 2)) * PW, *mineB = mineA + 8 * PW;
      if ((lane & 3) == 0) { mineA[0] = mxA; mineA[1] = lA; mineB[0] = mxB; mineB[1] = lB; }
#pragma unroll
      for (int nt = 0; nt < HD / 8; ++nt) {
        int d = 2 + 8 * nt + 2 * (lane & 3);
        mineA[d] = o[nt][0]; mineA[d + 1] = o[nt][1];
        mineB[d] = o[nt][2]; mineB[d + 1] = o[nt][3];
      }
      __syncthreads();
      {
        constexpr int DPT = HD / 16;                 // output dims per thread
        const int row = threadIdx.x >> 4, d0 = (threadIdx.x & 15) * DPT;
        const int m = mt * 16 + row;
        if (m < M) {
          float mr = -INFINITY, lr = 0.f, acc[DPT];
#pragma unroll
          for (int i = 0; i < DPT; ++i) acc[i] = 0.f;
#pragma unroll
          for (int w = 0; w < WARPS; ++w) {
            const float *pc = mbuf + ((size_t)w * 16 + row) * PW;
            float mn, a, b;
            fold_scales(mr, pc[0], mn, a, b);
            lr = lr * a + pc[1] * b;
#pragma unroll
            for (int i = 0; i < DPT; ++i) acc[i] = acc[i] * a + pc[2 + d0 + i] * b;
            mr = mn;
          }
          const int r = g_begin + m % nr, head = kvh * g + m / nr;
          float *dst = p.part + (((size_t)r * p.H + head) * p.cap + c) * PW;
          if ((threadIdx.x & 15) == 0) { dst[0] = mr; dst[1] = lr; }
#pragma unroll
          for (int i = 0; i < DPT; ++i) dst[2 + d0 + i] = acc[i];
        }
      }
      __syncthreads();
    }
    g_begin = g_end;
  }
}

// Folds a row's chunks in ascending order and normalises.  One warp per (row, head).
template <int HD>
__global__ void attn_merge_kernel(const AttnParams p) {
  constexpr int PW = HD + 2, DPL = HD / 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x, head = blockIdx.y * (blockDim.x >> 5) + warp;
  if (head >= p.H) return;
  const int nv = p.lin_end[r] + p.seg_len[r];
  const int nc = (nv + CH - 1) / CH;
  const float *src = p.part + ((size_t)r * p.H + head) * p.cap * PW;
  float m = -INFINITY, l = 0.f, acc[DPL];
#pragma unroll
  for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
  for (int c = 0; c < nc; ++c) {
    const float *pc = src + (size_t)c * PW;
    float mn, a, b;
    fold_scales(m, pc[0], mn, a, b);
    l = l * a + pc[1] * b;
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[i] = acc[i] * a + pc[2 + lane + 32 * i] * b;
    m = mn;
  }
  const float inv = 1.0f / l;
#pragma unroll
  for (int i = 0; i < DPL; ++i) p.out[(size_t)r * p.H * HD + head * HD + lane + 32 * i] = __float2bfloat16_rn(acc[i] * inv);
}

template <int HD>
size_t chunk_smem() { return (size_t)2 * CH * HD * 2 + (size_t)WARPS * 16 * (HD + 2) * 4 + OURO_MAX_ROWS * 4; }

}  // namespace

bool attention_tc_supported(const ouro_model_desc &d) { return d.dtype == OURO_BF16 && (d.head_dim == 64 || d.head_dim == 128); }

size_t attention_tc_scratch_bytes(const ouro_model_desc &d) {
  if (!attention_tc_supported(d)) return 0;
  size_t cap = (d.max_seq + CH - 1) / CH;
  return (size_t)OURO_MAX_ROWS * d.n_heads * cap * (d.head_dim + 2) * sizeof(float);
}

int attention_tc_setup() {
  if (cudaFuncSetAttribute(attn_chunk_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)chunk_smem<128>()) != cudaSuccess)
    return OURO_ECUDA;
  if (cudaFuncSetAttribute(attn_chunk_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)chunk_smem<64>()) != cudaSuccess)
    return OURO_ECUDA;
  return OURO_OK;
}

// n_vis_max: the largest number of visible keys over the block's rows (cache length + rows at most).
void launch_attention_tc(const ouro_model_desc &d, const void *q, const void *k_cache, const void *v_cache, const BlockDev &b,
                         int rows, int L, int n_vis_max, int layer, float *part, void *out, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  OURO_COUNT_LAUNCH();
  AttnParams p;
  size_t off = (size_t)layer * d.max_seq * d.n_kv_heads * d.head_dim;
  p.q = (const __nv_bfloat16 *)q;
  p.k = (const __nv_bfloat16 *)k_cache + off;
  p.v = (const __nv_bfloat16 *)v_cache + off;
  p.lin_end = b.lin_end; p.seg_start = b.seg_start; p.seg_len = b.seg_len; p.group = b.group;
  p.rows = rows; p.H = d.n_heads; p.Hkv = d.n_kv_heads; p.L = L;
  p.cap = (d.max_seq + CH - 1) / CH;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)d.head_dim);
  p.part = part;
  p.out = (__nv_bfloat16 *)out;
  dim3 grid((n_vis_max + CH - 1) / CH, d.n_kv_heads), mgrid(rows, (d.n_heads + 3) / 4);
  if (d.head_dim == 128) {
    attn_chunk_kernel<128><<<grid, THREADS, chunk_smem<128>(), s>>>(p);
    attn_merge_kernel<128><<<mgrid, 128, 0, s>>>(p);
  } else {
    attn_chunk_kernel<64><<<grid, THREADS, chunk_smem<64>(), s>>>(p);
    attn_merge_kernel<64><<<mgrid, 128, 0, s>>>(p);
  }
}
