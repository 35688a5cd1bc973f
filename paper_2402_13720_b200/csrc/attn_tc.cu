// Candidate-masked attention over the KV cache for a block of query rows (bf16, tensor cores, split along keys).
//
// Section 3.2 of the paper verifies K lengthened drafts in one forward by masking attention so that a phrase
// suffix sees the prefix, the draft and itself only (Eq. 8).  Here that mask is never materialised: a row is
// described by the number of keys it sees and by where its last keys live (its own candidate's cache slots),
// and the kernel maps "virtual positions" 0..n_vis-1 to cache slots on the fly.
//
// Work split.  Keys are cut by virtual position into aligned spans of 512; one CTA handles one (kv head, span)
// for up to 64 query rows (rows x query heads of the group; further rows go to further CTAs, which find the same
// keys in L2), so every cached byte is read from HBM once.  The CTA
// walks its span in chunks of 128 keys: K and V rows of the next chunk stream into a second shared-memory
// buffer (cp.async) while the current one is used.  Per chunk: the 8 warps split the keys for S = Q K^T
// (mma.sync), agree on each row's chunk maximum through shared memory, write P = exp2(S - max) as bf16 to shared
// memory, then split the head dimension for O += P V.  Running (max, sum, O) are kept per row across the chunks
// of the span; a second kernel folds the spans of a row in ascending order and normalises.
//
// Chunks below the cache length are the same for all rows.  A chunk holding the block's own keys differs
// between the trunk and each candidate: it is processed once per group, with that group's keys swapped into the
// tile and the other rows masked out (an exact no-op for them).  The value computed for a query depends only on
// (virtual position -> key) and on fixed chunk, span and warp boundaries, never on the other rows of the block:
// a token gets bit-identical attention whether it is verified inside a candidate block or decoded alone.
#include "ouro_internal.h"

// Optional timeline (compile with -DOURO_TRACE): see gemm_tc.cu.
#ifdef OURO_TRACE
__device__ unsigned long long g_attn_tc_trace[512][8];
__device__ __forceinline__ unsigned long long attn_tc_trace_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
  return t;
}
#define TRACE(slot) do { const int cta_ = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x; if (threadIdx.x == 0 && cta_ < 512) g_attn_tc_trace[cta_][slot] = attn_tc_trace_now(); } while (0)
extern "C" int ouro_trace_read_attn_tc(unsigned long long *out_host) {
  return (int)cudaMemcpyFromSymbol(out_host, g_attn_tc_trace, sizeof(g_attn_tc_trace));
}
#else
#define TRACE(slot) do { } while (0)
#endif

namespace {

constexpr int CH = 128;            // keys per chunk
constexpr int SC = 4;              // chunks per span
constexpr int SPAN = CH * SC;
constexpr int WARPS = 8;
constexpr int KW = CH / WARPS;     // keys per warp in the S phase (two 8-key MMA tiles)
constexpr int THREADS = WARPS * 32;
// Query rows per round: MT row tiles of 16 (MT = 4: 64 rows, or MT = 1: 16 rows for short blocks such as a draft
// model's single-row steps).  The kernel's loops over row tiles are unrolled, and with four tiles its machine code is
// 150 KB, of which a block with one live tile still walks most: a pass over a chunk then takes 4.3 us waiting for
// instruction fetches.  A row's arithmetic does not involve its tile's index or the other rows, so both sizes give the
// same bits.

struct AttnParams {
  const __nv_bfloat16 *q;          // [rows][H*HD] rotated queries
  const __nv_bfloat16 *k, *v;      // this layer's cache: [max_seq][Hkv*HD]
  const int32_t *lin_end, *seg_start, *seg_len, *group;
  int rows, H, Hkv, L, cap;        // L: cache length before the block; cap: span slots per (row, head)
  float scale_log2;
  float *part;                     // [rows][H][cap][HD+2]: max (log2 domain), sum, unnormalised output
  __nv_bfloat16 *out;              // [rows][H*HD]
  int direct;                      // every row's keys lie in span 0: the span kernel normalises and writes `out` itself
  const int *rows_dev;             // NULL, or the block's true row count in device memory (`rows` is then an upper bound)
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void cp_wait_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2_t(uint32_t addr, uint32_t &r0, uint32_t &r1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
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

// Dense query-row index m -> (block row, query head inside the kv group).  Groups are contiguous row ranges;
// group G with rows [a, b) owns the indices [g*a, g*b), ordered head-major inside the group.
__device__ __forceinline__ void map_row(int m, int g, int rows, const int *grp, int &row, int &hq) {
  int a = 0;
  while (true) {
    int b = a + 1;
    while (b < rows && grp[b] == grp[a]) ++b;
    if (m < g * b || b >= rows) {
      int e = m - g * a, n = b - a;
      hq = e / n;
      row = a + e % n;
      return;
    }
    a = b;
  }
}

template <int HD, int MT>
struct Smem {
  static constexpr int QR = 16 * MT;
  static constexpr int ROWB = HD * 2;                              // bytes per K/V/Q tile row
  static constexpr int KV = CH * ROWB;                             // one K or V buffer
  static constexpr int OFF_V = 2 * KV;                             // K[2] then V[2]
  static constexpr int OFF_Q = 4 * KV;
  static constexpr int OFF_P = OFF_Q + QR * ROWB;                  // P: [MT][16][CH] bf16
  static constexpr int OFF_WMAX = OFF_P + MT * 16 * CH * 2;        // [WARPS][QR]
  static constexpr int OFF_WSUM = OFF_WMAX + WARPS * QR * 4;
  static constexpr int OFF_NVIS = OFF_WSUM + WARPS * QR * 4;       // [OURO_MAX_ROWS]
  static constexpr int OFF_GRP = OFF_NVIS + OURO_MAX_ROWS * 4;
  static constexpr int OFF_MAP = OFF_GRP + OURO_MAX_ROWS * 4;      // [QR] block row | head << 16 of each query row
  static constexpr int BYTES = OFF_MAP + QR * 4;
};

template <int HD, int MT>
__global__ void __launch_bounds__(THREADS) attn_span_kernel(const AttnParams p) {
  using S = Smem<HD, MT>;
  constexpr int QR = S::QR;
  constexpr int CPR = HD / 8;                  // 16-byte pieces per row
  constexpr int ROWB = S::ROWB;
  constexpr int PW = HD + 2;
  constexpr int DW = HD / WARPS;               // output dims per warp in the P V phase (16 or 8)
  constexpr int NT2 = DW / 8;                  // 8-dim MMA tiles per warp
  extern __shared__ __align__(128) uint8_t smem[];
  float *wmax = (float *)(smem + S::OFF_WMAX), *wsum = (float *)(smem + S::OFF_WSUM);
  int *s_nvis = (int *)(smem + S::OFF_NVIS), *s_grp = (int *)(smem + S::OFF_GRP), *s_map = (int *)(smem + S::OFF_MAP);
  const uint32_t sm_u = smem_u32(smem);

  pdl_trigger();
  TRACE(0);
  // Everything up to pdl_wait() reads only what was complete before the forward pass began: the block description
  // (written by the assembling kernel, which is not launched programmatically and so has finished) and cache rows
  // below the cache length.  The queries and the block's own K/V rows come from the kernel just before this one.
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sc = blockIdx.x, kvh = blockIdx.y;
  const int g = p.H / p.Hkv, dkv = p.Hkv * HD;
  const int rows = p.rows_dev ? min(p.rows, __ldg(p.rows_dev)) : p.rows;   // written before the forward pass began
  const int M_all = g * rows;

  int nv_max = 0;
  for (int r = threadIdx.x; r < rows; r += THREADS) {
    s_nvis[r] = p.lin_end[r] + p.seg_len[r];
    s_grp[r] = p.group[r];
  }
  __syncthreads();
  for (int r = 0; r < rows; ++r) nv_max = max(nv_max, s_nvis[r]);
  const int span0 = sc * SPAN;
  const int n_chunks = min(SC, (nv_max - span0 + CH - 1) / CH);       // chunks of this span anybody sees

  // Stages the part of chunk ci every row shares (virtual positions below the cache length) and zeroes the rest.
  auto stage_common = [&](int ci, int buf) {
    const int c0 = span0 + ci * CH;
    for (int idx = threadIdx.x; idx < CH * CPR; idx += THREADS) {
      int row = idx / CPR, ch = idx % CPR, pos = c0 + row;
      uint32_t off = buf * S::KV + row * ROWB + ((ch ^ (row & 7)) << 4);
      if (pos < p.L) {
        size_t src = (size_t)pos * dkv + kvh * HD + ch * 8;
        cp_async16(sm_u + off, p.k + src);
        cp_async16(sm_u + S::OFF_V + off, p.v + src);
      } else {
        *reinterpret_cast<uint4 *>(smem + off) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4 *>(smem + S::OFF_V + off) = make_uint4(0, 0, 0, 0);
      }
    }
    cp_commit();
  };

  {
    // ---------------------------------------------------------------- this CTA's round of up to 64 query rows
    const int m0 = blockIdx.z * QR;
    // Query rows are ordered group by group (a group's rows for head 0, then for head 1, ..), so that the 64 rows
    // of a round belong to few groups and the chunk that holds block keys needs few passes.  Rows of this thread
    // in row tile mt: lane/4 and +8.
    if (threadIdx.x < QR) {
      int r0 = 0, hq = 0;
      if (m0 + (int)threadIdx.x < M_all) map_row(m0 + threadIdx.x, g, rows, s_grp, r0, hq);
      s_map[threadIdx.x] = r0 | (hq << 16);
    }
    __syncthreads();
    int nv[2 * MT], gr[2 * MT], rr[2 * MT], hh[2 * MT];
    bool any_row = false;
#pragma unroll
    for (int i = 0; i < 2 * MT; ++i) {
      int ml = (i >> 1) * 16 + (lane >> 2) + (i & 1) * 8;
      rr[i] = 0; hh[i] = kvh * g; nv[i] = 0; gr[i] = -1;
      if (m0 + ml < M_all) {
        rr[i] = s_map[ml] & 0xffff;
        hh[i] = kvh * g + (s_map[ml] >> 16);
        nv[i] = s_nvis[rr[i]];
        gr[i] = s_grp[rr[i]];
      }
      any_row = any_row || nv[i] > span0;
    }
    if (!__syncthreads_or(any_row)) return;            // nobody in this round reaches the span
    const int n_mt = (min(QR, M_all - m0) + 15) >> 4;  // row tiles that hold query rows; the others are skipped

    stage_common(0, 0);                                 // chunk 0 (its rows below the cache length) is on its way ...
    TRACE(1);
    pdl_wait();                                         // ... while the previous kernel finishes
    TRACE(2);
    for (int idx = threadIdx.x; idx < QR * CPR; idx += THREADS) {
      int row = idx / CPR, ch = idx % CPR, m = m0 + row;
      uint32_t off = S::OFF_Q + row * ROWB + ((ch ^ (row & 7)) << 4);
      if (m < M_all)
        cp_async16(sm_u + off, p.q + (size_t)(s_map[row] & 0xffff) * p.H * HD + (kvh * g + (s_map[row] >> 16)) * HD + ch * 8);
      else
        *reinterpret_cast<uint4 *>(smem + off) = make_uint4(0, 0, 0, 0);
    }
    cp_commit();                                        // Q is a group of its own, younger than chunk 0

    float o[MT][NT2][4], m_run[2 * MT], l_run[2 * MT];
#pragma unroll
    for (int i = 0; i < 2 * MT; ++i) { m_run[i] = -INFINITY; l_run[i] = 0.f; }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT2; ++nt) o[mt][nt][0] = o[mt][nt][1] = o[mt][nt][2] = o[mt][nt][3] = 0.f;

    for (int ci = 0; ci < n_chunks; ++ci) {
      const int buf = ci & 1, c0 = span0 + ci * CH;
      if (ci + 1 < n_chunks) { stage_common(ci + 1, buf ^ 1); cp_wait_but_one(); } else { cp_wait_all(); }
      __syncthreads();
      if (ci == 0) TRACE(3);
      const bool common = c0 + CH <= p.L;
      int g_begin = 0;
      while (g_begin < rows) {
        // -------------------------------------------------------------- one pass over the chunk
        int g_end = rows, gid = -2;                  // gid -2: every row takes part
        if (!common) {
          gid = s_grp[g_begin];
          g_end = g_begin + 1;
          while (g_end < rows && s_grp[g_end] == gid) ++g_end;
          const int last = g_end - 1, nvg = s_nvis[last];
          int lin_g = INT_MAX, seg_g = 0;
          if (p.seg_len[last] > 0) { lin_g = p.lin_end[last]; seg_g = p.seg_start[last]; }
          bool mine = false;
#pragma unroll
          for (int i = 0; i < 2 * MT; ++i) mine = mine || (gr[i] == gid && nv[i] > c0);
          if (!__syncthreads_or(mine)) { g_begin = g_end; continue; }   // no row of this round in the group
          // swap in the group's own keys: virtual positions [max(c0, L), min(c0 + CH, nvg))
          for (int idx = threadIdx.x; idx < CH * CPR; idx += THREADS) {
            int row = idx / CPR, ch = idx % CPR, pos = c0 + row;
            if (pos >= p.L && pos < nvg) {
              int slot = pos < lin_g ? pos : seg_g + (pos - lin_g);
              uint32_t off = buf * S::KV + row * ROWB + ((ch ^ (row & 7)) << 4);
              size_t src = (size_t)slot * dkv + kvh * HD + ch * 8;
              cp_async16(sm_u + off, p.k + src);
              cp_async16(sm_u + S::OFF_V + off, p.v + src);
            }
          }
          cp_commit();
          cp_wait_all();
          __syncthreads();
        }
        // row tiles none of whose rows takes part in this pass are left alone (same decision in every warp)
        bool live[MT];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
          live[mt] = mt < n_mt && (gid == -2 || __ballot_sync(0xffffffffu, gr[2 * mt] == gid || gr[2 * mt + 1] == gid) != 0);
        // ---- S = Q K^T for this warp's 16 keys, all row tiles
        float s[MT][2][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) s[mt][nt][0] = s[mt][nt][1] = s[mt][nt][2] = s[mt][nt][3] = 0.f;
        const uint32_t k_u = sm_u + buf * S::KV, v_u = sm_u + S::OFF_V + buf * S::KV;
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
          const int mi = lane >> 3;
          uint32_t b0, b1, b2, b3;
          {
            int row = warp * KW + (lane & 7) + ((mi >> 1) << 3), ch = 2 * ks + (mi & 1);
            ldsm_x4(k_u + row * ROWB + ((ch ^ (row & 7)) << 4), b0, b1, b2, b3);
          }
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            if (!live[mt]) continue;
            uint32_t a[4];
            int row = mt * 16 + (lane & 7) + ((mi & 1) << 3), ch = 2 * ks + (mi >> 1);
            ldsm_x4(sm_u + S::OFF_Q + row * ROWB + ((ch ^ (row & 7)) << 4), a[0], a[1], a[2], a[3]);
            mma16816(s[mt][0], a, b0, b1);
            mma16816(s[mt][1], a, b2, b3);
          }
        }
        // ---- mask by virtual position and group; warp-local row maxima (log2 domain)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          if (!live[mt]) continue;
          const int iA = 2 * mt, iB = 2 * mt + 1;
          const int nA = (gid == -2 || gr[iA] == gid) ? nv[iA] : 0, nB = (gid == -2 || gr[iB] == gid) ? nv[iB] : 0;
          float mxA = -INFINITY, mxB = -INFINITY;
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) {
            int kp = c0 + warp * KW + 8 * nt + 2 * (lane & 3);
            s[mt][nt][0] = kp < nA ? s[mt][nt][0] * p.scale_log2 : -INFINITY;
            s[mt][nt][1] = kp + 1 < nA ? s[mt][nt][1] * p.scale_log2 : -INFINITY;
            s[mt][nt][2] = kp < nB ? s[mt][nt][2] * p.scale_log2 : -INFINITY;
            s[mt][nt][3] = kp + 1 < nB ? s[mt][nt][3] * p.scale_log2 : -INFINITY;
            mxA = fmaxf(mxA, fmaxf(s[mt][nt][0], s[mt][nt][1]));
            mxB = fmaxf(mxB, fmaxf(s[mt][nt][2], s[mt][nt][3]));
          }
          mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 1));
          mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 2));
          mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 1));
          mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 2));
          if ((lane & 3) == 0) {
            wmax[(mt * 16 + (lane >> 2)) * WARPS + warp] = mxA;
            wmax[(mt * 16 + (lane >> 2) + 8) * WARPS + warp] = mxB;
          }
        }
        __syncthreads();
        // ---- new running maximum, P = exp2(S - max) to shared memory, warp-local row sums
        float scale_old[2 * MT];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          if (!live[mt]) { scale_old[2 * mt] = scale_old[2 * mt + 1] = 1.f; continue; }
#pragma unroll
          for (int hb = 0; hb < 2; ++hb) {
            const int i = 2 * mt + hb, row = mt * 16 + (lane >> 2) + 8 * hb;
            const float4 m0v = *reinterpret_cast<const float4 *>(wmax + row * WARPS);
            const float4 m1v = *reinterpret_cast<const float4 *>(wmax + row * WARPS + 4);
            const float mc = fmaxf(fmaxf(fmaxf(m0v.x, m0v.y), fmaxf(m0v.z, m0v.w)), fmaxf(fmaxf(m1v.x, m1v.y), fmaxf(m1v.z, m1v.w)));
            const float mn = fmaxf(m_run[i], mc);
            scale_old[i] = (m_run[i] == -INFINITY) ? 0.f : exp2f(m_run[i] - mn);   // mn finite whenever m_run is
            m_run[i] = mn;
            const float use = mn == -INFINITY ? 0.f : mn;
            float sum = 0.f;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
              float p0 = exp2f(s[mt][nt][2 * hb] - use), p1 = exp2f(s[mt][nt][2 * hb + 1] - use);
              sum += p0 + p1;
              int ch = warp * 2 + nt;                               // 16-byte piece: keys 8*ch .. 8*ch+7
              uint32_t off = S::OFF_P + (mt * 16 + (row & 15)) * (CH * 2) + ((ch ^ (row & 7)) << 4) + 4 * (lane & 3);
              *reinterpret_cast<uint32_t *>(smem + off) = pack_bf16(p0, p1);
            }
            sum += __shfl_xor_sync(0xffffffffu, sum, 1);
            sum += __shfl_xor_sync(0xffffffffu, sum, 2);
            if ((lane & 3) == 0) wsum[row * WARPS + warp] = sum;
          }
        }
        __syncthreads();
        // ---- running sums and O = O * scale + P V for this warp's slice of the head dimension
#pragma unroll
        for (int i = 0; i < 2 * MT; ++i) {
          if (!live[i >> 1]) continue;
          const int row = (i >> 1) * 16 + (lane >> 2) + 8 * (i & 1);
          const float4 s0 = *reinterpret_cast<const float4 *>(wsum + row * WARPS);
          const float4 s1 = *reinterpret_cast<const float4 *>(wsum + row * WARPS + 4);
          const float add = ((((((s0.x + s0.y) + s0.z) + s0.w) + s1.x) + s1.y) + s1.z) + s1.w;    // warp order
          l_run[i] = l_run[i] * scale_old[i] + add;
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int nt = 0; nt < NT2; ++nt) {
            o[mt][nt][0] *= scale_old[2 * mt]; o[mt][nt][1] *= scale_old[2 * mt];
            o[mt][nt][2] *= scale_old[2 * mt + 1]; o[mt][nt][3] *= scale_old[2 * mt + 1];
          }
#pragma unroll
        for (int kk = 0; kk < CH / 16; ++kk) {
          const int mi = lane >> 3;
          uint32_t b0, b1, b2 = 0, b3 = 0;
          if (NT2 == 2) {
            int row = 16 * kk + (lane & 7) + ((mi & 1) << 3), ch = warp * 2 + (mi >> 1);
            ldsm_x4_t(v_u + row * ROWB + ((ch ^ (row & 7)) << 4), b0, b1, b2, b3);
          } else {
            int row = 16 * kk + (lane & 7) + ((mi & 1) << 3), ch = warp;
            ldsm_x2_t(v_u + row * ROWB + ((ch ^ (row & 7)) << 4), b0, b1);
          }
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            if (!live[mt]) continue;
            uint32_t a[4];
            int row = (lane & 7) + ((mi & 1) << 3), ch = 2 * kk + (mi >> 1);
            ldsm_x4(sm_u + S::OFF_P + (mt * 16 + row) * (CH * 2) + ((ch ^ (row & 7)) << 4), a[0], a[1], a[2], a[3]);
            mma16816(o[mt][0], a, b0, b1);
            if (NT2 == 2) mma16816(o[mt][NT2 - 1], a, b2, b3);
          }
        }
        __syncthreads();                              // wmax, wsum, P and the tile may change now
        g_begin = g_end;
      }
    }
    TRACE(4);
    // ---- the span's piece of every row of the round that reaches it
#pragma unroll
    for (int i = 0; i < 2 * MT; ++i) {
      if (nv[i] <= span0) continue;
      if (p.direct) {
        // what the merge kernel would compute from this single span: weight exp2(0) = 1, then o * (1 / l)
        const float inv = 1.0f / l_run[i];
#pragma unroll
        for (int nt = 0; nt < NT2; ++nt) {
          int d = warp * DW + 8 * nt + 2 * (lane & 3);
          *reinterpret_cast<__nv_bfloat162 *>(p.out + ((size_t)rr[i] * p.H + hh[i]) * HD + d) =
              __floats2bfloat162_rn(o[i >> 1][nt][2 * (i & 1)] * inv, o[i >> 1][nt][2 * (i & 1) + 1] * inv);
        }
        continue;
      }
      float *dst = p.part + (((size_t)rr[i] * p.H + hh[i]) * p.cap + sc) * PW;
      if (warp == 0 && (lane & 3) == 0) { dst[0] = m_run[i]; dst[1] = l_run[i]; }
#pragma unroll
      for (int nt = 0; nt < NT2; ++nt) {
        int d = warp * DW + 8 * nt + 2 * (lane & 3);
        *reinterpret_cast<float2 *>(dst + 2 + d) = make_float2(o[i >> 1][nt][2 * (i & 1)], o[i >> 1][nt][2 * (i & 1) + 1]);
      }
    }
    TRACE(5);
  }
}

}  // namespace

bool attention_tc_supported(const ouro_model_desc &d) {
  return d.dtype == OURO_BF16 && (d.head_dim == 64 || d.head_dim == 128) && d.max_seq <= 32 * SPAN;   // the fold looks at one span per lane
}

size_t attention_tc_scratch_bytes(const ouro_model_desc &d) {
  if (!attention_tc_supported(d)) return 0;
  size_t cap = (d.max_seq + SPAN - 1) / SPAN;
  return (size_t)OURO_MAX_ROWS * d.n_heads * cap * (d.head_dim + 2) * sizeof(float);
}

template <int HD, int MT>
static bool tc_prepare() {
  return cudaFuncSetAttribute(attn_span_kernel<HD, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<HD, MT>::BYTES) == cudaSuccess;
}
int attention_tc_setup() {
  return tc_prepare<128, 4>() && tc_prepare<128, 1>() && tc_prepare<64, 4>() && tc_prepare<64, 1>() ? OURO_OK : OURO_ECUDA;
}

// n_vis_max: an upper bound of the number of keys any row of the block sees (cache length + rows).
bool launch_attention_tc(const ouro_model_desc &d, const void *q, const void *k_cache, const void *v_cache, const BlockDev &b,
                         int rows, int L, int n_vis_max, int layer, float *part, void *out, const int *rows_dev, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  AttnParams p;
  p.rows_dev = rows_dev;
  size_t off = (size_t)layer * d.max_seq * d.n_kv_heads * d.head_dim;
  p.q = (const __nv_bfloat16 *)q;
  p.k = (const __nv_bfloat16 *)k_cache + off;
  p.v = (const __nv_bfloat16 *)v_cache + off;
  p.lin_end = b.lin_end; p.seg_start = b.seg_start; p.seg_len = b.seg_len; p.group = b.group;
  p.rows = rows; p.H = d.n_heads; p.Hkv = d.n_kv_heads; p.L = L;
  p.cap = (d.max_seq + SPAN - 1) / SPAN;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)d.head_dim);
  p.part = part;
  p.out = (__nv_bfloat16 *)out;
  const int m_all = (d.n_heads / d.n_kv_heads) * rows;      // query rows per kv head, served 64 per CTA
  const int mt = m_all <= 16 ? 1 : 4, qr = 16 * mt;         // rows per round (m_all is an upper bound when the count is on the device)
  dim3 grid((n_vis_max + SPAN - 1) / SPAN, d.n_kv_heads, (m_all + qr - 1) / qr);
  p.direct = n_vis_max <= SPAN;                             // a single span: nothing to fold
  if (d.head_dim == 128) {
    if (mt == 1) launch_pdl(attn_span_kernel<128, 1>, grid, THREADS, Smem<128, 1>::BYTES, s, p);
    else launch_pdl(attn_span_kernel<128, 4>, grid, THREADS, Smem<128, 4>::BYTES, s, p);
  } else {
    if (mt == 1) launch_pdl(attn_span_kernel<64, 1>, grid, THREADS, Smem<64, 1>::BYTES, s, p);
    else launch_pdl(attn_span_kernel<64, 4>, grid, THREADS, Smem<64, 4>::BYTES, s, p);
  }
  return !p.direct;
}
