// Candidate-masked attention on the sm_100a tensor cores (tcgen05 + TMEM, K/V tiles fetched by TMA), head dim 128.
//
// Same contract as the mma.sync kernel next door: Section 3.2 of the paper verifies K lengthened drafts in one
// forward under a mask in which a phrase suffix sees the prefix, the draft and itself (Eq. 8); a row is described
// by the number of keys it sees and by where its last keys live, and keys are addressed by "virtual position".
//
// Work split.  Keys are cut by virtual position into aligned spans of 512; one CTA handles one (span, kv head)
// for a round of up to 128 query rows (block rows x query heads of the group, ordered group by group).  It walks
// the span in chunks of 128 keys.  Per chunk:
//     S = Q K^T      one 128 x 128 x 128 tcgen05 contraction into TMEM (Q and K K-major in 128-byte swizzle),
//     softmax        the threads of query row t read its 128 scores from TMEM, mask by virtual position, keep a
//                    running (max, sum) and write P = exp2(S - max) as bf16 to shared memory,
//     O_c = P V      a second contraction (V is the MN-major operand, straight from the cache layout),
//     O = O a + O_c  in registers of the row's threads.
// Warp 0 fetches the tiles (TMA, two stages of K and V), warp 1 issues the contractions, warps 2-9 are the row
// threads, two per query row: one for keys 0-63 of a chunk and dims 0-63 of the output, one for the upper halves.
// S and O_c are double buffered in TMEM so that the scores of the next pass are computed while the current one's
// softmax runs.
//
// A chunk that holds the block's own keys is processed once per group (trunk, each candidate), each pass with a
// tile of its own: cache slots equal virtual positions for the prefix and the trunk, so the tile the TMA fetched
// is already right for them; for a candidate, warp 0 copies its suffix rows over the tile before the pass (the
// tile is fetched once per stage; what an earlier candidate left in rows beyond a pass's own keys is masked).
// Rows of other groups sit the pass out.
// The value computed for a query depends only on (virtual position -> key) and on the fixed chunk and span
// boundaries, never on the other rows of the block: a token gets bit-identical attention whether it is verified
// inside a candidate block or decoded alone.
//
// Every mbarrier wait is bounded; on expiry the CTA raises the context's status word, stops waiting and drains.
#include <cuda.h>

#include "ouro_internal.h"

// Optional timeline (compile with -DOURO_TRACE): see gemm_tc.cu.
#ifdef OURO_TRACE
__device__ unsigned long long g_attn_trace[512][8];
__device__ __forceinline__ unsigned long long attn_trace_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
  return t;
}
#define TRACE(slot) do { const int cta_ = blockIdx.y * gridDim.x + blockIdx.x; if (cta_ < 512) g_attn_trace[cta_][slot] = attn_trace_now(); } while (0)
extern "C" int ouro_trace_read_attn(unsigned long long *out_host) {
  return (int)cudaMemcpyFromSymbol(out_host, g_attn_trace, sizeof(g_attn_trace));
}
#else
#define TRACE(slot) do { } while (0)
#endif

namespace {

constexpr int HD = 128;
constexpr int CH = 128;            // keys per chunk
constexpr int SC = 4;              // chunks per span
constexpr int SPAN = CH * SC;      // must equal the span of the merge kernel
constexpr int QR = 128;            // query rows per round = TMEM lanes
constexpr int PW = HD + 2;
constexpr int ROW_THREADS = 256;  // two threads per query row
constexpr int THREADS = 64 + ROW_THREADS;
constexpr uint32_t SPIN_LIMIT = 1u << 22;

constexpr int HALF = 128 * 128;    // bytes of a [128 rows][64 bf16] half tile in 128-byte swizzle
constexpr int TILE = 2 * HALF;     // [2 halves][128 rows][128 B]
constexpr int OFF_Q = 0;
constexpr int OFF_K = OFF_Q + TILE;          // two stages
constexpr int OFF_V = OFF_K + 2 * TILE;      // two stages
constexpr int OFF_P = OFF_V + 2 * TILE;      // two buffers
constexpr int OFF_MISC = OFF_P + 2 * TILE;
constexpr int MAX_ITEMS = SC * 33;
constexpr int MAX_GROUPS = 32;

struct Misc {
  uint64_t full[2], empty[2], s_ready[2], p_ready[2], o_ready[2], patched[2];
  uint32_t tmem_base;
  int abort_flag, n_items, n_groups;
  int wcnt[4];
  int gs[MAX_GROUPS + 2];   // first row of each group, then the row count
  int gmax[MAX_GROUPS];     // keys seen by the round's rows of each group (maximum)
  int lin[128], len[128];   // lin_end and seg_len of every block row
  int map[QR];              // tile row -> block row | head << 8 | group ordinal << 16, or -1
  int items[MAX_ITEMS];
};
constexpr int SMEM_BYTES = OFF_MISC + 3072;
static_assert(sizeof(Misc) <= 3072, "misc area");

// work item: chunk | group ordinal (63: every row) << 3 | flags
enum { IT_PATCH = 1 << 9, IT_REUSE = 1 << 10 };   // REUSE: the stage already holds this chunk's tile

struct TmParams {
  CUtensorMap kmap, vmap;          // [layers * max_seq][Hkv * HD] bf16, box 64 x 128, 128-byte swizzle
  const __nv_bfloat16 *q;          // [rows][H*HD] rotated queries
  const __nv_bfloat16 *k, *v;      // this layer's cache: [max_seq][Hkv*HD]
  const int32_t *lin_end, *seg_start, *seg_len, *group;
  int rows, H, Hkv, L, cap, row0;  // row0: first row of this layer in the tensor maps
  int n_spans;
  float scale_log2;
  float *part;                     // [rows][H][cap][HD+2]: max (log2 domain), sum, unnormalised output
  __nv_bfloat16 *out;              // [rows][H*HD], written here only when `direct`
  int direct;                      // every row's keys lie in span 0: normalise and write `out`, no folding needed
  int *status;
  const int *rows_dev;             // NULL, or the block's true row count in device memory (`rows` is then an upper bound)
  const uint8_t *pf_ptr[3];        // regions to bring into L2 for the kernels that follow (see L2Prefetch); each CTA asks
  uint32_t pf_bytes[3];            // for an equal share of every region
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  False when the limit ran out or another thread of the CTA has given up; the first thread to
// give up raises the status word.  After that nobody in the CTA blocks any more.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, Misc *ms, int *status) {
  for (uint32_t i = 0; i < SPIN_LIMIT; ++i) {
    if (mbar_test(bar, parity)) return true;
    if ((i & 63) == 63 && *(volatile int *)&ms->abort_flag) return false;
  }
  if (atomicExch(&ms->abort_flag, 1) == 0) atomicExch(status, 1);
  return false;
}
// The cache rows are read once per forward pass: marked evict-first in L2, so that they do not push out the weights
// prefetched for the kernels that follow.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint64_t *bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;" ::"r"(dst),
      "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "l"(0x12F0000000000000ull)
      : "memory");
}
// K-major operand in 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t desc_k(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
// MN-major operand in 128-byte swizzle: 64 contiguous elements of the MN dimension per 128-byte row, 8 rows (K
// indices) per 1024-byte atom; atoms along K are 1024 bytes apart, the next 64 MN elements HALF bytes further.
__device__ __forceinline__ uint64_t desc_mn(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFF) >> 4) | ((uint64_t)(HALF >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
__device__ __forceinline__ void mma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Issues the load of 32 columns of this warp's lane quarter.  The values arrive asynchronously: they may be used
// after tmem_ld_wait32() has been applied to the same array (it waits for every load issued so far and ties the
// registers to the wait, so that the compiler keeps their uses behind it).
__device__ __forceinline__ void tmem_ld32_issue(uint32_t addr, float *v) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
               : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]), "=f"(v[8]), "=f"(v[9]), "=f"(v[10]), "=f"(v[11]), "=f"(v[12]), "=f"(v[13]), "=f"(v[14]), "=f"(v[15]), "=f"(v[16]), "=f"(v[17]), "=f"(v[18]), "=f"(v[19]), "=f"(v[20]), "=f"(v[21]), "=f"(v[22]), "=f"(v[23]), "=f"(v[24]), "=f"(v[25]), "=f"(v[26]), "=f"(v[27]), "=f"(v[28]), "=f"(v[29]), "=f"(v[30]), "=f"(v[31])
               : "r"(addr));
}
__device__ __forceinline__ void tmem_ld_wait32(float *v) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+f"(v[0]), "+f"(v[1]), "+f"(v[2]), "+f"(v[3]), "+f"(v[4]), "+f"(v[5]), "+f"(v[6]), "+f"(v[7]), "+f"(v[8]), "+f"(v[9]), "+f"(v[10]), "+f"(v[11]), "+f"(v[12]), "+f"(v[13]), "+f"(v[14]), "+f"(v[15]), "+f"(v[16]), "+f"(v[17]), "+f"(v[18]), "+f"(v[19]), "+f"(v[20]), "+f"(v[21]), "+f"(v[22]), "+f"(v[23]), "+f"(v[24]), "+f"(v[25]), "+f"(v[26]), "+f"(v[27]), "+f"(v[28]), "+f"(v[29]), "+f"(v[30]), "+f"(v[31])
               :
               : "memory");
}
// 16 columns, issued and waited for.
__device__ __forceinline__ void tmem_ld16(uint32_t addr, float *v) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
               : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]), "=f"(v[8]), "=f"(v[9]), "=f"(v[10]), "=f"(v[11]), "=f"(v[12]), "=f"(v[13]), "=f"(v[14]), "=f"(v[15])
               : "r"(addr));
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+f"(v[0]), "+f"(v[1]), "+f"(v[2]), "+f"(v[3]), "+f"(v[4]), "+f"(v[5]), "+f"(v[6]), "+f"(v[7]), "+f"(v[8]), "+f"(v[9]), "+f"(v[10]), "+f"(v[11]), "+f"(v[12]), "+f"(v[13]), "+f"(v[14]), "+f"(v[15])
               :
               : "memory");
}
__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// 2^x for x <= 0 on the special-function unit (results below the normal range become zero).
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&t);
}

constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);  // fp32 += bf16 x bf16, 128 x 128
constexpr uint32_t IDESC_PV = IDESC_S | (1u << 16);                                                            // B operand MN-major

__global__ void __launch_bounds__(THREADS, 1) attn_tm_kernel(const __grid_constant__ TmParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sm_u = smem_u32(smem);
  Misc *ms = reinterpret_cast<Misc *>(smem + OFF_MISC);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // blockIdx.x walks (span, kv head) with the last span of every head first: it holds the block's own keys and
  // takes one pass per group, so it should not be what the grid ends on
  const int sc = p.n_spans - 1 - blockIdx.x / p.Hkv, kvh = blockIdx.x % p.Hkv, m0 = blockIdx.y * QR;
  const int rows = p.rows_dev ? min(p.rows, __ldg(p.rows_dev)) : p.rows;   // written before the forward pass began
  const int g = p.H / p.Hkv, dkv = p.Hkv * HD, M_all = g * rows, span0 = sc * SPAN;

  if (tid == 0) TRACE(0);
  if (tid == 32) {
    // the weights the next kernels start with do not depend on anything computed here: ask for this CTA's share now
    const uint32_t u = blockIdx.y * gridDim.x + blockIdx.x, U = gridDim.x * gridDim.y;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
      const uint32_t bytes = p.pf_bytes[r];
      if (bytes == 0) continue;
      const uint32_t share = ((bytes + U - 1) / U + 15u) & ~15u, off = u * share;
      if (off < bytes)
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p.pf_ptr[r] + off), "r"(min(share, bytes - off)) : "memory");
    }
  }
  if (sm_u & 1023) {                                   // the swizzled tiles need a 1024-byte aligned base
    if (tid == 0) atomicExch(p.status, 1);
    return;
  }
  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&ms->full[i], 1);
      mbar_init(&ms->empty[i], 1);
      mbar_init(&ms->s_ready[i], 1);
      mbar_init(&ms->p_ready[i], ROW_THREADS);
      mbar_init(&ms->o_ready[i], 1);
      mbar_init(&ms->patched[i], 1);
    }
    ms->abort_flag = 0;
    ms->n_items = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < MAX_GROUPS) ms->gmax[tid] = 0;
  if (warp == 1) {                                     // S and O_c, double buffered: all 512 columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ms->tmem_base)), "r"(512u));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  pdl_trigger();
  // Everything up to pdl_wait() reads only what was complete before the forward pass began: the block description
  // (written by the assembling kernel, which is not launched programmatically and so has finished) and cache rows
  // below the cache length.  The queries and the block's own K/V rows come from the kernel just before this one.

  // ---- groups are contiguous row ranges: find their first rows (warps 0-3, one block row per thread)
  bool start = false;
  unsigned bal = 0;
  if (tid < 128) {
    int lin = 0, len = 0;
    if (tid < rows) {
      start = tid == 0 || p.group[tid] != p.group[tid - 1];
      lin = p.lin_end[tid];
      len = p.seg_len[tid];
    }
    ms->lin[tid] = lin;
    ms->len[tid] = len;
    bal = __ballot_sync(0xffffffffu, start);
    if (lane == 0) ms->wcnt[warp] = __popc(bal);
  }
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  if (tid < 128) {
    int ord = __popc(bal & ((1u << lane) - 1));
    for (int w = 0; w < warp; ++w) ord += ms->wcnt[w];
    if (start && ord < MAX_GROUPS) ms->gs[ord] = tid;
    if (tid == 0) {
      int n = min(ms->wcnt[0] + ms->wcnt[1] + ms->wcnt[2] + ms->wcnt[3], MAX_GROUPS);
      ms->n_groups = n;
      ms->gs[n] = rows;
    }
  }
  __syncthreads();
  // ---- tile row t holds query row m0 + (t % 32) * 4 + t / 32 of the group-major order, which spreads a short
  //      round over the four softmax warps
  if (tid < QR) {
    const int m = m0 + (tid & 31) * 4 + (tid >> 5);
    int info = -1;
    if (m < M_all) {
      const int ng = ms->n_groups;
      int o = 0;
      while (o + 1 < ng && m >= g * ms->gs[o + 1]) ++o;
      const int a = ms->gs[o], n = ms->gs[o + 1] - a, e = m - g * a;
      const int r = a + e % n, hq = e / n;
      info = r | (hq << 8) | (o << 16);
      atomicMax(&ms->gmax[o], ms->lin[r] + ms->len[r]);
    }
    ms->map[tid] = info;
  }
  __syncthreads();
  // ---- the work items of this CTA, in order: (chunk, group) passes
  if (tid == 0) {
    const int ng = ms->n_groups;
    int rmax = 0, n = 0;
    for (int o = 0; o < ng; ++o) rmax = max(rmax, ms->gmax[o]);
    if (rmax > span0) {
      const int nch = min(SC, (rmax - span0 + CH - 1) / CH);
      for (int ci = 0; ci < nch; ++ci) {
        const int c0 = span0 + ci * CH;
        if (c0 + CH <= p.L) {
          ms->items[n++] = ci | (63 << 3);
        } else {
          // the chunk's tile is fetched into both stages once; later passes only patch their rows over it
          int in_chunk = 0;
          for (int o = 0; o < ng; ++o) {
            if (ms->gmax[o] <= c0) continue;
            const int last = ms->gs[o + 1] - 1, len = ms->len[last], lin = ms->lin[last];
            const bool patch = len > 0 && lin < c0 + CH && lin + len > c0;
            ms->items[n++] = ci | (o << 3) | (patch ? IT_PATCH : 0) | (in_chunk >= 2 ? IT_REUSE : 0);
            ++in_chunk;
          }
        }
      }
    }
    ms->n_items = n;
  }
  __syncthreads();
  // ---- every pass gets a K/V stage of its own (pass i: stage i % 2); tiles of chunks wholly below the cache
  //      length can start streaming in before the previous kernel has finished
  auto request_tile = [&](int i, int ci) {
    const int st = i & 1;
    mbar_expect_tx(&ms->full[st], 2 * TILE);
    const int x = kvh * HD, y = p.row0 + span0 + ci * CH;
    tma_load_2d(sm_u + OFF_K + st * TILE, &p.kmap, &ms->full[st], x, y);
    tma_load_2d(sm_u + OFF_K + st * TILE + HALF, &p.kmap, &ms->full[st], x + 64, y);
    tma_load_2d(sm_u + OFF_V + st * TILE, &p.vmap, &ms->full[st], x, y);
    tma_load_2d(sm_u + OFF_V + st * TILE + HALF, &p.vmap, &ms->full[st], x + 64, y);
  };
  int early = 0;                                       // passes whose tile was requested before the wait
  if (warp == 0) {
    const int n = ms->n_items;
    while (early < 2 && early < n && ((ms->items[early] >> 3) & 63) == 63) {
      if (lane == 0) request_tile(early, ms->items[early] & 7);
      ++early;
    }
  }
  if (tid == 0) TRACE(1);
  pdl_wait();
  if (tid == 0) TRACE(2);
  // ---- Q tile: K-major, two halves of 64 dims, 128-byte swizzle; rows without a query are zero
  {
    // every thread's pieces are requested before the first is stored: one round trip to L2 instead of one per piece
    constexpr int QI = (QR * 16 + THREADS - 1) / THREADS;
    uint4 val[QI];
#pragma unroll
    for (int i = 0; i < QI; ++i) {
      const int idx = tid + i * THREADS, t = idx >> 4, ch = idx & 15;
      val[i] = make_uint4(0, 0, 0, 0);
      if (idx < QR * 16) {
        const int info = ms->map[t];
        if (info >= 0) {
          const int r = info & 0xff, hq = (info >> 8) & 0xff;
          val[i] = __ldg(reinterpret_cast<const uint4 *>(p.q + ((size_t)r * p.H + kvh * g + hq) * HD + ch * 8));
        }
      }
    }
#pragma unroll
    for (int i = 0; i < QI; ++i) {
      const int idx = tid + i * THREADS, t = idx >> 4, ch = idx & 15;
      if (idx < QR * 16)
        *reinterpret_cast<uint4 *>(smem + OFF_Q + (ch >> 3) * HALF + t * 128 + (((ch & 7) ^ (t & 7)) << 4)) = val[i];
    }
  }
  fence_async_smem();
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const int n_items = ms->n_items;
  const uint32_t tmem = ms->tmem_base;

  if (n_items > 0) {
    if (warp == 0) {
      // ================================================================ tile producer (TMA; whole warp for the patches)
      // (a wait that gives up raises the abort flag and the status word itself; nobody blocks after that)
      for (int i = 0; i < n_items; ++i) {
        const int it = ms->items[i], ci = it & 7, go = (it >> 3) & 63, st = i & 1;
        if (i >= early) {
          if (i >= 2) mbar_wait(&ms->empty[st], ((i >> 1) - 1) & 1, ms, p.status);
          if (lane == 0) {
            if (it & IT_REUSE) mbar_arrive(&ms->full[st]);   // nothing to fetch: the phase completes at once
            else request_tile(i, ci);
          }
        }
        if (it & IT_PATCH) {
          // a candidate's pass: its suffix rows go over the tile the TMA fetched (slots = positions up to the trunk)
          mbar_wait(&ms->full[st], (i >> 1) & 1, ms, p.status);
          const int c0 = span0 + ci * CH, last = ms->gs[go + 1] - 1;
          const int lin_g = ms->lin[last], seg_g = p.seg_start[last], len_g = ms->len[last];
          const int lo = max(c0, lin_g), hi = min(c0 + CH, lin_g + len_g);
          for (int idx = lane; idx < (hi - lo) * 32; idx += 32) {
            const int pos = lo + (idx >> 5), w = idx & 31, ch = w & 15, trow = pos - c0;
            const size_t src = (size_t)(seg_g + pos - lin_g) * dkv + kvh * HD + ch * 8;
            const uint4 val = *reinterpret_cast<const uint4 *>(((w >> 4) ? p.v : p.k) + src);
            *reinterpret_cast<uint4 *>(smem + ((w >> 4) ? OFF_V : OFF_K) + st * TILE + (ch >> 3) * HALF + trow * 128 +
                                       (((ch & 7) ^ (trow & 7)) << 4)) = val;
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(&ms->patched[st]);
        }
      }
      // nothing of this CTA may still be in flight when it leaves: wait (bounded) for the last tile of each stage
      if (lane == 0) {
        for (int st = 0; st < 2; ++st) {
          const int n_st = (n_items + 1 - st) >> 1;        // tiles requested into this stage
          if (n_st == 0) continue;
          const uint32_t par = (n_st - 1) & 1;
          for (uint32_t spin = 0; spin < SPIN_LIMIT && !mbar_test(&ms->full[st], par); ++spin) {}
        }
      }
    } else if (warp == 1) {
      // ================================================================ contraction issue
      if (lane == 0) {
        bool issued = false;
        uint32_t patch_par = 0;                        // bit st: parity of the next patched tile of stage st
        auto issue_s = [&](int i) {
          const uint64_t da = desc_k(sm_u + OFF_Q), db = desc_k(sm_u + OFF_K + (i & 1) * TILE);
          const uint32_t d = tmem + (i & 1) * 128;
#pragma unroll
          for (int ks = 0; ks < HD / 16; ++ks) {
            const uint32_t off = ((ks >> 2) * HALF + (ks & 3) * 32) >> 4;   // the address field counts 16-byte units
            mma_bf16(d, da + off, db + off, IDESC_S, ks > 0);
          }
          mma_commit(&ms->s_ready[i & 1]);
        };
        // the tile of pass i is complete: fetched, and patched where the pass needs it
        auto tile_ready = [&](int i) {
          const int st = i & 1;
          if (!mbar_test(&ms->full[st], (i >> 1) & 1)) return false;
          if ((ms->items[i] & IT_PATCH) && !mbar_test(&ms->patched[st], (patch_par >> st) & 1)) return false;
          return true;
        };
        auto tile_taken = [&](int i) {
          if (ms->items[i] & IT_PATCH) patch_par ^= 1u << (i & 1);
        };
        for (int i = 0; i < n_items; ++i) {
          const int st = i & 1, b = i & 1;
          if (!issued) {
            bool ready = false;
            for (uint32_t spin = 0; spin < SPIN_LIMIT && !ready; ++spin) {
              ready = tile_ready(i);
              if ((spin & 63) == 63 && *(volatile int *)&ms->abort_flag) break;
            }
            if (!ready) {
              if (atomicExch(&ms->abort_flag, 1) == 0) atomicExch(p.status, 1);
            }
            tile_taken(i);
            fence_after_sync();
            issue_s(i);
          }
          issued = false;
          // while P of this pass is being made: the scores of the next pass, as soon as its tile is there
          bool want = i + 1 < n_items, p_done = false;
          for (uint32_t spin = 0; spin < SPIN_LIMIT && !p_done; ++spin) {
            if (want && tile_ready(i + 1)) {
              tile_taken(i + 1);
              fence_after_sync();
              issue_s(i + 1);
              issued = true;
              want = false;
            }
            p_done = mbar_test(&ms->p_ready[b], (i >> 1) & 1);
            if ((spin & 63) == 63 && *(volatile int *)&ms->abort_flag) break;
          }
          if (!p_done) {
            if (atomicExch(&ms->abort_flag, 1) == 0) atomicExch(p.status, 1);
          }
          fence_after_sync();
          {
            const uint64_t da = desc_k(sm_u + OFF_P + b * TILE), dv = desc_mn(sm_u + OFF_V + st * TILE);
            const uint32_t d = tmem + 256 + b * 128;
#pragma unroll
            for (int kk = 0; kk < CH / 16; ++kk)
              mma_bf16(d, da + (((kk >> 2) * HALF + (kk & 3) * 32) >> 4), dv + ((kk * 2048) >> 4), IDESC_PV, kk > 0);
          }
          mma_commit(&ms->o_ready[b]);
          mma_commit(&ms->empty[st]);
        }
      }
    } else {
      // ================================================================ the row threads, two per query row
      // Thread (t, h) of tile row t: h = 0 owns keys 0-63 of a chunk's scores and dims 0-63 of the output, h = 1
      // the upper halves.  Both find the row maximum over all 128 scores, so they agree on it without talking.
      const int h = (warp - 2) >> 2;
      const int t = 32 * (warp & 3) + lane;            // TMEM lane = tile row; a warp reaches its own quarter only
      const uint32_t lane_addr = tmem + ((uint32_t)(32 * (warp & 3)) << 16);
      const int info = ms->map[t];
      const bool has = info >= 0;
      const int r = has ? (info & 0xff) : 0, hq = has ? ((info >> 8) & 0xff) : 0, my_o = has ? (info >> 16) : -1;
      const int nv = has ? ms->lin[r] + ms->len[r] : 0;
      float m_run = -INFINITY, l_run = 0.f, alpha_prev = 1.f;
      float o_reg[HD / 2];
#pragma unroll
      for (int i = 0; i < HD / 2; ++i) o_reg[i] = 0.f;
      bool pending = false, act_prev = false;

      auto accumulate = [&](int i) {                   // O = O * alpha + O_c of pass i
        mbar_wait(&ms->o_ready[i & 1], (i >> 1) & 1, ms, p.status);
        fence_after_sync();
        if (__any_sync(0xffffffffu, act_prev)) {        // TMEM loads are warp-wide: every lane takes part
          float v[64];
          tmem_ld32_issue(lane_addr + 256 + (i & 1) * 128 + h * 64, v);
          tmem_ld32_issue(lane_addr + 256 + (i & 1) * 128 + h * 64 + 32, v + 32);
          tmem_ld_wait32(v);
          tmem_ld_wait32(v + 32);
          if (act_prev) {
#pragma unroll
            for (int j = 0; j < 64; ++j) o_reg[j] = o_reg[j] * alpha_prev + v[j];
          }
        }
        pending = false;
      };

      for (int i = 0; i < n_items; ++i) {
        const int it = ms->items[i], ci = it & 7, go = (it >> 3) & 63, b = i & 1;
        const int c0 = span0 + ci * CH;
        const bool active = has && nv > c0 && (go == 63 || go == my_o);
        mbar_wait(&ms->s_ready[b], (i >> 1) & 1, ms, p.status);
        if (i == 0 && tid == 64) TRACE(3);
        fence_after_sync();
        float alpha = 1.f;
        const int nk = active ? min(nv - c0, CH) : 0;  // keys of this chunk the row sees: tile columns below nk
        const int nk_w = __reduce_max_sync(0xffffffffu, nk);
        const bool whole = __all_sync(0xffffffffu, !active || nk >= CH);   // no score of an active row is masked
        // Both forms below compute the same numbers for a row, in the same order (four interleaved partial sums
        // over ascending keys; a masked key adds an exact zero), so which one a warp takes - that depends on its
        // other rows - never shows in a row's result.  TMEM loads are warp-wide: every lane takes part in them.
        uint8_t *prow = smem + OFF_P + b * TILE + h * HALF + t * 128;     // this thread's 128 bytes of P
        float mn = m_run, sum = 0.f;
        if (whole) {
          // ---- row maximum over the chunk (scaling by a positive factor commutes with max, bit for bit)
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            float vm[64];
            tmem_ld32_issue(lane_addr + b * 128 + hh * 64, vm);
            tmem_ld32_issue(lane_addr + b * 128 + hh * 64 + 32, vm + 32);
            tmem_ld_wait32(vm);
            tmem_ld_wait32(vm + 32);
#pragma unroll
            for (int j = 0; j < 64; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], vm[j]);
          }
          mn = fmaxf(m_run, fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2);
          // ---- P = exp2(S - max) for this thread's 64 keys
          float v[64];
          tmem_ld32_issue(lane_addr + b * 128 + h * 64, v);
          tmem_ld32_issue(lane_addr + b * 128 + h * 64 + 32, v + 32);
          tmem_ld_wait32(v);
          tmem_ld_wait32(v + 32);
          if (active) {
            float sum4[4] = {0.f, 0.f, 0.f, 0.f};
            uint32_t w[32];
#pragma unroll
            for (int j = 0; j < 64; j += 2) {
              const float p0 = ex2(v[j] * p.scale_log2 - mn), p1 = ex2(v[j + 1] * p.scale_log2 - mn);
              sum4[j & 3] += p0;
              sum4[(j & 3) + 1] += p1;
              w[j >> 1] = pack_bf16(p0, p1);
            }
            sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
#pragma unroll
            for (int q8 = 0; q8 < 8; ++q8)              // 16-byte piece q8 of key half h: keys 64 h + 8 q8 ..
              *reinterpret_cast<uint4 *>(prow + ((q8 ^ (t & 7)) << 4)) = make_uint4(w[4 * q8], w[4 * q8 + 1], w[4 * q8 + 2], w[4 * q8 + 3]);
          }
        } else if (nk_w > 0) {
          // a chunk that ends inside the block's own keys: only the 16-key pieces below nk_w are looked at
          const int npc = (nk_w + 15) >> 4;
          float mxv = -INFINITY;
          for (int pc = 0; pc < npc; ++pc) {
            float v[16];
            tmem_ld16(lane_addr + b * 128 + pc * 16, v);
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (pc * 16 + j < nk) mxv = fmaxf(mxv, v[j]);
          }
          mn = fmaxf(m_run, mxv * p.scale_log2);       // finite for an active row: it sees key c0 at least
          float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int q = 0; q < 4; ++q) {                 // the four 16-key pieces of this thread's half
            const int pc = 4 * h + q;
            uint32_t w[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) w[j] = 0u;
            if (pc < npc) {
              float v[16];
              tmem_ld16(lane_addr + b * 128 + pc * 16, v);
              if (active) {
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                  const float p0 = (pc * 16 + j < nk) ? ex2(v[j] * p.scale_log2 - mn) : 0.f;
                  const float p1 = (pc * 16 + j + 1 < nk) ? ex2(v[j + 1] * p.scale_log2 - mn) : 0.f;
                  sum4[j & 3] += p0;
                  sum4[(j & 3) + 1] += p1;
                  w[j >> 1] = pack_bf16(p0, p1);
                }
              }
            }
            if (active) {
              *reinterpret_cast<uint4 *>(prow + (((2 * q) ^ (t & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
              *reinterpret_cast<uint4 *>(prow + (((2 * q + 1) ^ (t & 7)) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
            }
          }
          sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        }
        if (active) {
          alpha = (m_run == -INFINITY) ? 0.f : ex2(m_run - mn);
          l_run = l_run * alpha + sum;
          m_run = mn;
        }
        fence_async_smem();
        fence_before_sync();
        mbar_arrive(&ms->p_ready[b]);
        if (pending) accumulate(i - 1);
        pending = true;
        act_prev = active;
        alpha_prev = alpha;
      }
      if (pending) accumulate(n_items - 1);
      if (tid == 64) TRACE(4);
      // ---- the span's piece of this row: the two halves of the row sum are added in a fixed order
      float *lsum = reinterpret_cast<float *>(smem + OFF_Q);      // Q is no longer read: every contraction has completed
      lsum[h * QR + t] = l_run;
      asm volatile("bar.sync 1, %0;" ::"n"(ROW_THREADS) : "memory");
      if (has && nv > span0 && p.direct) {
        // what the merge kernel would compute from this single span: weight exp2(0) = 1, then o * (1 / l)
        const float inv = 1.0f / (lsum[t] + lsum[QR + t]);
        __nv_bfloat16 *dst = p.out + ((size_t)r * p.H + kvh * g + hq) * HD + h * 64;
#pragma unroll
        for (int d = 0; d < HD / 2; d += 8) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) w[e] = pack_bf16(o_reg[d + 2 * e] * inv, o_reg[d + 2 * e + 1] * inv);
          *reinterpret_cast<uint4 *>(dst + d) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      } else if (has && nv > span0) {
        float *dst = p.part + (((size_t)r * p.H + kvh * g + hq) * p.cap + sc) * PW;
        if (h == 0) *reinterpret_cast<float2 *>(dst) = make_float2(m_run, lsum[t] + lsum[QR + t]);
#pragma unroll
        for (int d = 0; d < HD / 2; d += 2) *reinterpret_cast<float2 *>(dst + 2 + h * 64 + d) = make_float2(o_reg[d], o_reg[d + 1]);
      }
    }
  }
  fence_before_sync();
  __syncthreads();
  if (tid == 0) TRACE(5);
  if (warp == 1) {
    fence_after_sync();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u));
  }
}

}  // namespace

bool attention_tm_supported(const ouro_model_desc &d) {
  return d.dtype == OURO_BF16 && d.head_dim == HD && d.n_heads % d.n_kv_heads == 0 && d.n_heads / d.n_kv_heads <= 255 &&
         d.max_seq <= 32 * SPAN;              // the fold looks at one span per lane
}

int attention_tm_setup() {
  if (cudaFuncSetAttribute(attn_tm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess) return OURO_ECUDA;
  return OURO_OK;
}

// kmap / vmap: CUtensorMap objects over the whole K and V caches, [n_layers * max_seq][Hkv * 128] bf16 with a
// 64 x 128 box in 128-byte swizzle.  Returns true when the spans still have to be folded (attn_fold.cuh: by the kernel
// that consumes the attention output); with a single span the kernel has written `out` itself.
bool launch_attention_tm(const ouro_model_desc &d, const void *q, const void *kmap, const void *vmap, const void *k_cache,
                         const void *v_cache, const BlockDev &b, int rows, int L, int n_vis_max, int layer, float *part,
                         void *out, int *status, const int *rows_dev, const L2Prefetch &pf, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  TmParams p;
  for (int r = 0; r < 3; ++r) {
    const bool ok = pf.ptr[r] && pf.bytes[r] > 0 && pf.bytes[r] < (1ull << 31) && pf.bytes[r] % 16 == 0 && ((uintptr_t)pf.ptr[r] & 15) == 0;
    p.pf_ptr[r] = ok ? (const uint8_t *)pf.ptr[r] : nullptr;
    p.pf_bytes[r] = ok ? (uint32_t)pf.bytes[r] : 0u;
  }
  p.kmap = *reinterpret_cast<const CUtensorMap *>(kmap);
  p.vmap = *reinterpret_cast<const CUtensorMap *>(vmap);
  size_t off = (size_t)layer * d.max_seq * d.n_kv_heads * d.head_dim;
  p.q = (const __nv_bfloat16 *)q;
  p.k = (const __nv_bfloat16 *)k_cache + off;
  p.v = (const __nv_bfloat16 *)v_cache + off;
  p.lin_end = b.lin_end; p.seg_start = b.seg_start; p.seg_len = b.seg_len; p.group = b.group;
  p.rows = rows; p.H = d.n_heads; p.Hkv = d.n_kv_heads; p.L = L;
  p.cap = (d.max_seq + SPAN - 1) / SPAN;
  p.row0 = layer * d.max_seq;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)d.head_dim);
  p.part = part;
  p.out = (__nv_bfloat16 *)out;
  p.direct = n_vis_max <= SPAN;
  p.status = status;
  p.rows_dev = rows_dev;
  const int m_all = (d.n_heads / d.n_kv_heads) * rows;
  p.n_spans = (n_vis_max + SPAN - 1) / SPAN;
  dim3 grid(p.n_spans * d.n_kv_heads, (m_all + QR - 1) / QR);
  launch_pdl(attn_tm_kernel, grid, THREADS, SMEM_BYTES, s, p);
  return !p.direct;
}
