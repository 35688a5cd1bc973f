// Weight-streaming GEMM for a few dozen tokens on sm_100a tensor cores (tcgen05 + TMEM), fed by TMA.
//
//   Y[t, n] = sum_k X[t, k] * W[n, k]      X: [rows <= 128, K] bf16 activations, W: [N, K] bf16 weights
//
// The verification forward is bound by the one pass over the weights (the paper's premise: checking dozens
// of tokens costs about as much as one, Section 3.2), so the kernel is organised around the weight stream:
//   * operands are swapped: a 128-row slab of W is the MMA's M side, the tokens (padded to a multiple of 16)
//     are its N side; the fp32 accumulator [128 x T] lives in TMEM;
//   * one persistent CTA per SM; the (tile, k-block) iteration space is cut into equal contiguous spans
//     (stream-K), so every SM streams the same number of bytes whatever N and K are;
//   * a span that covers only part of a tile's K range leaves a partial tile in scratch memory.  After its last
//     MMA every contributor of a tile adds up a share of the tile's tokens (token t belongs to contributor
//     t mod n) in ascending K order and runs the epilogue on them.  A CTA waits for the others' partials only
//     after it has published all of its own, so the waits cannot form a cycle (and they are bounded); the
//     result does not depend on arrival order;
//   * warp 0 issues TMA loads into a ring of shared-memory stages (128-byte swizzle), warp 1 issues
//     tcgen05.mma and releases stages with tcgen05.commit, warps 2-5 drain TMEM (double buffered) and run the
//     epilogue: plain store, residual add, or SiLU(gate)*up for the stacked gate/up matrices.
// The span boundaries depend on N, K and the grid only, never on the number of rows, and an output element
// is a function of its own row of X: a token's result is bitwise the same in a 1-row and in a 128-row call.
// Every mbarrier wait is bounded; on expiry the CTA raises the context's status word and drains.
#include <cuda.h>

#include "ouro_internal.h"
#include "weight_stream.cuh"
#include "attn_fold.cuh"

void ouro_set_global_error(const std::string &msg);   // api.cu

// Optional timeline of the GEMM launches (compile with -DOURO_TRACE, see paper_2402_13720_b200/trace.py): selected
// threads of every CTA stamp the global nanosecond timer at fixed points; ouro_trace_read_gemm copies the stamps
// of the most recent launch of every kind out.  Compiled out by default.
#ifdef OURO_TRACE
__device__ unsigned long long g_gemm_trace[8][160][16];
__device__ __forceinline__ unsigned long long trace_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
  return t;
}
#define TRACE(slot) do { if (blockIdx.x < 160) g_gemm_trace[p.trace_id & 7][blockIdx.x][slot] = trace_now(); } while (0)
extern "C" int ouro_trace_read_gemm(unsigned long long *out_host) {
  return (int)cudaMemcpyFromSymbol(out_host, g_gemm_trace, sizeof(g_gemm_trace));
}
#else
#define TRACE(slot) do { } while (0)
#endif

namespace {

using ws::BLOCK_K;
using ws::TILE_N;
using ws::Span;
constexpr int A_BYTES = TILE_N * BLOCK_K * 2;
constexpr int THREADS = 224;      // warp 0 weight TMA, warp 1 MMA, warps 2..5 epilogue, warp 6 activation TMA
constexpr int W_PRODUCERS = 2;    // lanes of warp 0 that issue the weight copies, stage by stage in turn (a power of two, smaller than the ring)
constexpr int MAX_GRID = 160;
constexpr int SLOT_FLOATS = TILE_N * OURO_MAX_ROWS;
constexpr uint32_t SPIN_LIMIT = 1u << 24;
constexpr unsigned long long HINT_EVICT_FIRST = 0x12F0000000000000ull;
constexpr unsigned long long HINT_EVICT_LAST = 0x14F0000000000000ull;

enum { MODE_STORE = 0, MODE_RESIDUAL = 1, MODE_SWIGLU = 2, MODE_HEAD = 3, MODE_QKV = 4 };
// HEAD: per-tile row maxima (+ optional logits).  QKV: rotary positions on q and k, q to its buffer, k and v appended to the cache.

struct GemmParams {
  CUtensorMap a[3];   // weight matrices stacked along the output dimension (q|k|v), or gate and up
  CUtensorMap b;      // activations, box = 64 x t_pad
  int a_tiles[3];     // tiles of each stacked matrix (MODE_STORE / MODE_RESIDUAL)
  int a_rows[3];      // output features of each stacked matrix
  int a_count;
  int mode;
  int tiles;          // total tiles
  int kb;             // k-blocks per tile (K / 64)
  int t_pad;          // tokens padded to a multiple of 16 (MMA N)
  int rows;           // valid tokens (an upper bound when rows_dev is set)
  const int *rows_dev;  // NULL, or where the block's true row count sits in device memory: the host then sizes the
                        // launch for the largest block the decoding parameters allow and never reads the count
  int stages;
  float *out_f32;     // MODE_STORE / MODE_RESIDUAL: [rows, ldo]
  int ldo;
  __nv_bfloat16 *out_bf16;  // MODE_SWIGLU: [rows, F]
  float *tile_max;    // MODE_HEAD: [tiles][128] largest logit of each token inside the tile ...
  int *tile_arg;      //            ... and its vocabulary index (smallest index among equals)
  // RMSNorm folded into the GEMMs around it: g*x/rms(x) feeds a GEMM as bf16(g*x), and the per-token factor
  // 1/rms(x) multiplies that GEMM's output instead.  The producer of x (a residual-add epilogue) leaves bf16(g*x)
  // and, per 128-column tile, each token's sum of squares; the consumer adds the tile sums in order.
  // MODE_QKV: stacked q|k|v tiles hold whole heads (head_dim 64 or 128); pairs (i, i + head_dim/2) are rotated by
  // the row's position; q goes to q_out [rows, dq], k and v to cache slots L + row of this layer
  const int32_t *pos;
  const float *cos_t, *sin_t;   // [max_seq, head_dim/2]
  __nv_bfloat16 *q_out, *k_out, *v_out;
  int head_dim, dq, dkv, L;
  const __nv_bfloat16 *gain;  // MODE_RESIDUAL: gain of the norm that follows (NULL: plain residual add)
  __nv_bfloat16 *xb;          // MODE_RESIDUAL: bf16(gain * x_new), [rows, ldo]
  float *ss_out;              // MODE_RESIDUAL: [tiles][128] per-tile sums of squares of x_new
  const float *ss_in;         // other modes: sums of squares of the activation rows (NULL: no scaling)
  int ss_tiles;
  float ss_inv_d, eps;
  float *scratch;     // [grid][2][t][128] partial tiles
  int *counters;      // [tiles] partial tiles published, as (gen << 8) + count: a word left by an earlier GEMM is
                      // smaller than this GEMM's (gen << 8), so nothing has to be cleared between GEMMs or launches
  int gen;            // this GEMM's generation number (1 .. 2^22, grows with every GEMM the context runs)
  int *status;        // context status word
  int trace_id;           // which GEMM of the layer this is (timeline builds only)
  uint32_t wait_limit;    // polls of a partial-tile wait before it gives up (1 << 22 unless a test shortens it)
};

// A chain of GEMMs run by one persistent launch, each consuming what the one before produced (output projection ->
// gate/up -> down -> next layer's q,k,v or the LM head).  The weight producer runs straight on into the next GEMM's
// tiles; the activations of GEMM i + 1 are fetched once GEMM i has finished all its tiles, which the CTAs learn from
// a counter in global memory (one per chain position, counting finished tiles, never reset: the host passes the value
// it will have reached).  All GEMMs of a chain have the same rows / t_pad / stages.
constexpr int MAX_CHAIN = 4;
struct ChainParams {
  GemmParams g[MAX_CHAIN];
  int n;
  int *finished;            // [MAX_CHAIN + 1] tiles finished, per chain position (monotonic); last: CTAs done folding
  int target[MAX_CHAIN];    // value finished[i] has when GEMM i of this launch is complete
  // The first GEMM's activations may be the attention output, still in per-span pieces: every CTA first folds a share
  // of the (row, head) pairs, and the first activation tile is fetched once all CTAs have.
  fold::Params fold;
  int fold_target;                // value finished[MAX_CHAIN] has once every CTA has done its share of the work in front
  // ... or the embedding rows of the block's tokens (first layer): gathered by all CTAs the same way.
  struct Embed {
    const __nv_bfloat16 *table;   // [vocab][d]; NULL: nothing to gather
    const int32_t *tok;           // [rows]
    const __nv_bfloat16 *gain;    // first norm's gain [d]
    float *x;                     // residual stream [rows][d]
    __nv_bfloat16 *xb;            // bf16(gain * x) [rows][d]
    float *ss;                    // [d / 128][128] sums of squares per 128-column tile
    const int *rows_dev;
    int rows, d;
  } embed;
};
static_assert(sizeof(ChainParams) <= 4096, "kernel parameters");

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
// Bounded wait: false when the limit ran out or another warp of the CTA has given up (the caller raises the status
// word and drains).
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, uint32_t limit = SPIN_LIMIT) {
  uint32_t addr = smem_u32(bar);
  for (uint32_t i = 0; i < limit; ++i) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(addr), "r"(parity)
        : "memory");
    if (ok) return true;
    if ((i & 255) == 255 && abort_flag && *abort_flag) return false;
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y,
                                            unsigned long long hint) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4}], [%2], %5;" ::"r"(smem_u32(dst)),
      "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "l"(hint)
      : "memory");
}
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  // K-major operand in 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
  return (uint64_t)((addr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
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
__device__ __forceinline__ void tmem_ld16(uint32_t addr, float *v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(addr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// order-preserving map float -> uint32 (and back), so that integer max picks the largest float
__device__ __forceinline__ uint32_t ordered_u32(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ordered_f32(uint32_t u) {
  return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}
// x * sigmoid(x) with the fast exponential and reciprocal (the result is rounded to bf16 right after)
__device__ __forceinline__ float silu(float x) { return __fdividef(x, 1.0f + __expf(-x)); }
__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// one half (64 threads) of the epilogue warps; grp = 0 or 1
__device__ __forceinline__ void group_barrier(int grp) { asm volatile("bar.sync %0, 64;" ::"r"(2 + grp) : "memory"); }
constexpr int STAGE_TOK = 64;     // tokens of a whole tile parked in shared memory at a time
constexpr int STAGE_PITCH = TILE_N + 4;   // floats per parked token: 16-byte aligned rows that start 4 banks apart
constexpr int STAGE_BYTES = STAGE_TOK * STAGE_PITCH * 4;

// The schedule of this launch for CTA blockIdx.x (see weight_stream.cuh).
struct SpanWalker : ws::SpanWalker {
  __device__ SpanWalker(const GemmParams &p) : ws::SpanWalker(p.tiles, p.kb, (int)gridDim.x, (int)blockIdx.x) {}
};

// Locates a tile: which stacked matrix, its first row there, and the first output column.
__device__ __forceinline__ void locate(const GemmParams &p, int tile, int &seg, int &row0, int &col0, int &valid) {
  seg = 0;
  col0 = 0;
  int t = tile;
  while (seg + 1 < p.a_count && t >= p.a_tiles[seg]) {
    t -= p.a_tiles[seg];
    col0 += p.a_rows[seg];
    ++seg;
  }
  row0 = t * TILE_N;
  col0 += row0;
  valid = min(TILE_N, p.a_rows[seg] - row0);
}

// Bounded wait until GEMM `i` of the chain has finished all its tiles (acquire).
__device__ __forceinline__ bool counter_wait(const int *counter, int target, const int *status, uint32_t limit) {
  for (uint32_t spin = 0; spin < limit; ++spin) {
    int seen;
    asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
    if (seen - target >= 0) return true;
    if ((spin & 15) == 15 && *(volatile const int *)status != 0) return false;   // some CTA has given up: nobody waits on
  }
  return false;
}
__device__ __forceinline__ bool chain_wait(const ChainParams &cp, int i) {
  return counter_wait(cp.finished + i, cp.target[i], cp.g[0].status, 1u << 22);
}

__global__ void __launch_bounds__(THREADS, 1) gemm_tc_kernel(const __grid_constant__ ChainParams cp) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const GemmParams &p0 = cp.g[0];                 // rows, t_pad and stages are common to the chain
  const int n_stages = p0.stages;
  const int b_bytes = p0.t_pad * BLOCK_K * 2;
  const int stage_bytes = A_BYTES + b_bytes;
  uint8_t *ring = smem;
  float *xchg = (float *)(ring + (size_t)n_stages * stage_bytes);          // [64 tokens][128] accumulators of a whole tile
  uint64_t *bars = (uint64_t *)((uint8_t *)xchg + STAGE_BYTES);
  uint64_t *full = bars, *empty = bars + 16, *acc_full = bars + 32, *acc_empty = bars + 34;
  uint32_t *tmem_base_p = (uint32_t *)(bars + 36);
  volatile int *abort_flag = (volatile int *)(bars + 37);
  volatile int *wait_flag = (volatile int *)(bars + 39);   // [0..1]: outcome of an accumulator wait; [2]: a fix-up gave up; [4..5]: outcome of a fix-up group's wait
  uint64_t *drain_bar = bars + 44;                          // give-up path: "every contraction issued so far has completed"
  float *rs = (float *)(bars + 48);                         // [128] per-token factor 1/rms of the consumed activations
  int *spos = (int *)(rs + OURO_MAX_ROWS);                  // [128] token positions (rotary table rows), QKV epilogue

  pdl_trigger();
  if (threadIdx.x == 0) { const GemmParams &p = p0; TRACE(0); }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int acc_cols = p0.t_pad <= 32 ? 32 : p0.t_pad <= 64 ? 64 : 128;   // columns per accumulator buffer

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(&full[s], 2);          // weight producer + activation producer, each with its byte count
      mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&acc_full[a], 1);
      mbar_init(&acc_empty[a], 4);
    }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_p)),
                 "r"((uint32_t)(2 * acc_cols)));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_base_p;
  uint32_t n_issued = 0;                           // producer lanes: stages they have issued copies into

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane < W_PRODUCERS) {
      // The weights do not depend on the previous kernel, so this warp never waits for it: the ring fills with
      // weight tiles while the predecessor drains.  The activation tiles come from warp 6, after its wait.
      // One thread runs this loop once per 16 KB stage; at 40 GB/s per SM that is every 0.4 us, so the loop carries
      // no division and nothing that is constant over a span: stage index and ring round are counted along.
      uint32_t n = 0, round = 0;
      int st = 0;
      bool ok = true;
      for (int ci = 0; ci < cp.n && ok; ++ci) {
      const GemmParams &p = cp.g[ci];
      const bool swiglu = p.mode == MODE_SWIGLU;
      SpanWalker w(p);
      Span s;
      while (ok && w.next(s)) {
        int seg = 0, row0 = s.tile * 64, col0, valid;
        if (!swiglu) locate(p, s.tile, seg, row0, col0, valid);
        const CUtensorMap *m0 = &p.a[seg];
        uint8_t *sa = ring + (size_t)st * stage_bytes;
        for (int kb = s.kb0; kb < s.kb1; ++kb, ++n) {
          if ((n & (W_PRODUCERS - 1)) == (uint32_t)lane) {           // the lanes take the stages in turn
            if (round > 0) {
              ok = mbar_wait(&empty[st], (round - 1) & 1, abort_flag) && !*abort_flag;
              if (!ok) break;
            }
            mbar_expect_tx(&full[st], A_BYTES);
            if (swiglu) {
              tma_load_2d(sa, &p.a[0], &full[st], kb * BLOCK_K, row0, HINT_EVICT_FIRST);
              tma_load_2d(sa + A_BYTES / 2, &p.a[1], &full[st], kb * BLOCK_K, row0, HINT_EVICT_FIRST);
            } else {
              tma_load_2d(sa, m0, &full[st], kb * BLOCK_K, row0, HINT_EVICT_FIRST);
            }
          }
          sa += stage_bytes;
          if (++st == n_stages) { st = 0; ++round; sa = ring; }
        }
      }
      TRACE(8);
      }
      if (!ok) { *abort_flag = 1; atomicExch(p0.status, 1); }
      n_issued = n;
    }
  } else if (warp == 6) {
    // ---------------------------------------------------------------- activation producer
    if (lane == 0) {
      pdl_wait();                                  // the first GEMM's activations are the previous kernel's output
      uint32_t n = 0, round = 0;
      int st = 0;
      uint8_t *sb = ring + A_BYTES;
      bool ok = true;
      if (cp.fold.part || cp.embed.table) {        // ... once every CTA has done its share of the fold / the gather
        ok = counter_wait(cp.finished + MAX_CHAIN, cp.fold_target, p0.status, 1u << 22);
        asm volatile("fence.proxy.async;" ::: "memory");
      }
      for (int ci = 0; ci < cp.n && ok; ++ci) {
        const GemmParams &p = cp.g[ci];
        if (ci > 0) {
          // they are what the GEMM before this one wrote: wait until all its tiles are finished, then make
          // those generic-proxy writes visible to the copy engine's reads
          ok = chain_wait(cp, ci - 1) && !*abort_flag;
          if (!ok) break;
          asm volatile("fence.proxy.async;" ::: "memory");
        }
        TRACE(1);
        SpanWalker w(p);
        Span s;
        while (ok && w.next(s)) {
          for (int kb = s.kb0; kb < s.kb1; ++kb, ++n) {
            if (round > 0) {
              ok = mbar_wait(&empty[st], (round - 1) & 1, abort_flag) && !*abort_flag;
              if (!ok) break;
            }
            mbar_expect_tx(&full[st], b_bytes);
            tma_load_2d(sb, &p.b, &full[st], kb * BLOCK_K, 0, HINT_EVICT_LAST);
            sb += stage_bytes;
            if (++st == n_stages) { st = 0; ++round; sb = ring + A_BYTES; }
          }
        }
      }
      if (!ok) { *abort_flag = 1; atomicExch(p0.status, 1); }
      n_issued = n;
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p0.t_pad >> 3) << 17) | ((uint32_t)(TILE_N >> 4) << 24);
      uint32_t n = 0, item = 0, round = 0;
      int st = 0;
      uint32_t sa = smem_u32(ring);
      const uint32_t ring0 = sa;
      bool ok = true;
      for (int ci = 0; ci < cp.n && ok; ++ci) {
      const GemmParams &p = cp.g[ci];
      SpanWalker w(p);
      Span s;
      bool first = true;
      while (ok && w.next(s)) {
        int a = item & 1;
        if (item >= 2) ok = mbar_wait(&acc_empty[a], ((item >> 1) - 1) & 1, abort_flag) && !*abort_flag;
        if (!ok) break;
        fence_after_sync();
        uint32_t tmem_d = tmem_base + a * acc_cols;
        for (int kb = s.kb0; kb < s.kb1; ++kb, ++n) {
          ok = mbar_wait(&full[st], round & 1, abort_flag) && !*abort_flag;
          if (!ok) break;
          if (first) { TRACE(2); first = false; }
          fence_after_sync();
          const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sa + A_BYTES);
#pragma unroll
          for (int k = 0; k < BLOCK_K / 16; ++k) mma_bf16(tmem_d, da + 2 * k, db + 2 * k, idesc, (kb > s.kb0 || k > 0) ? 1u : 0u);
          mma_commit(&empty[st]);
          sa += stage_bytes;
          if (++st == n_stages) { st = 0; ++round; sa = ring0; }
        }
        if (!ok) break;
        mma_commit(&acc_full[a]);
        ++item;
      }
      TRACE(3);
      }
      if (!ok) { *abort_flag = 1; atomicExch(p0.status, 1); }
    }
  } else {
    // ---------------------------------------------------------------- epilogue warps
    pdl_wait();
    const int q = warp & 3;                      // TMEM lane quarter this warp may read
    const int nl = q * 32 + lane;                // row of the tile held by this thread
    const int et = threadIdx.x - 64;             // 0..127 among the epilogue threads
    uint32_t item = 0;
    bool ok = true;
    float v[16];
    if (cp.fold.part || cp.embed.table) {
      const int gw = (int)blockIdx.x * 4 + (warp - 2), nw = (int)gridDim.x * 4;
      if (cp.fold.part) {
        fold::run(cp.fold, gw, nw, lane);
      } else {
        // Embedding rows into the residual stream, plus what the first norm's consumer needs: bf16(gain * x) and the
        // sums of squares per 128-column tile.  One warp per (row, tile): four columns per lane.
        const ChainParams::Embed &e = cp.embed;
        const int rows = e.rows_dev ? min(e.rows, __ldg(e.rows_dev)) : e.rows, tiles = (e.d + TILE_N - 1) / TILE_N;
        for (int it = gw; it < rows * tiles; it += nw) {
          const int r = it / tiles, col = (it - r * tiles) * TILE_N + 4 * lane;
          float sq = 0.f;
          if (col < e.d) {                                            // d is a multiple of 64: four columns are in or out together
            const uint2 raw = __ldg(reinterpret_cast<const uint2 *>(e.table + (size_t)__ldg(e.tok + r) * e.d + col));
            const uint2 graw = __ldg(reinterpret_cast<const uint2 *>(e.gain + col));
            const __nv_bfloat162 a01 = *reinterpret_cast<const __nv_bfloat162 *>(&raw.x), a23 = *reinterpret_cast<const __nv_bfloat162 *>(&raw.y);
            const __nv_bfloat162 g01 = *reinterpret_cast<const __nv_bfloat162 *>(&graw.x), g23 = *reinterpret_cast<const __nv_bfloat162 *>(&graw.y);
            const float v[4] = {__low2float(a01), __high2float(a01), __low2float(a23), __high2float(a23)};
            const float gv[4] = {__low2float(g01), __high2float(g01), __low2float(g23), __high2float(g23)};
            *reinterpret_cast<float4 *>(e.x + (size_t)r * e.d + col) = make_float4(v[0], v[1], v[2], v[3]);
            __nv_bfloat162 lo = __floats2bfloat162_rn(gv[0] * v[0], gv[1] * v[1]), hi = __floats2bfloat162_rn(gv[2] * v[2], gv[3] * v[3]);
            *reinterpret_cast<uint2 *>(e.xb + (size_t)r * e.d + col) = make_uint2(*(uint32_t *)&lo, *(uint32_t *)&hi);
            sq = (v[0] * v[0] + v[1] * v[1]) + (v[2] * v[2] + v[3] * v[3]);
          }
#pragma unroll
          for (int o = 16; o; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
          if (lane == 0) e.ss[(size_t)(it - r * tiles) * OURO_MAX_ROWS + r] = sq;
        }
      }
      __threadfence();
      epi_barrier();
      if (et == 0) atomicAdd(cp.finished + MAX_CHAIN, 1);
      if (cp.embed.table) {
        // the first GEMM's per-token factors are sums over what ALL CTAs gathered
        if (et == 0) wait_flag[0] = counter_wait(cp.finished + MAX_CHAIN, cp.fold_target, p0.status, 1u << 22) && !*abort_flag;
        epi_barrier();
        ok = wait_flag[0] != 0;
        epi_barrier();
        __threadfence();
      }
    }
    for (int ci = 0; ci < cp.n && ok; ++ci) {
    const GemmParams &p = cp.g[ci];
    const bool publish = ci + 1 < cp.n;          // a later GEMM of the chain consumes this one's output
    const int rows = p.rows_dev ? min(p.rows, __ldg(p.rows_dev)) : p.rows;
    SpanWalker w(p);
    Span s;
    int pend_tile[2], pend_n[2], pend_first[2], n_pend = 0;     // partial tiles this CTA contributed to (<= 2)
    float *stage = xchg;                                         // [STAGE_TOK tokens][STAGE_PITCH] fp32, 128 tile rows each

    // Finishing tokens of a tile.  Whatever produced the accumulator values - this CTA's own whole tile, parked
    // in shared memory token-major, or the partial tiles of all contributors in scratch - the last step is the
    // same: a group of G threads walks over "its" tokens, a warp's 32 lanes holding the tile's 128 rows (= output
    // columns) four apiece, so every global access is a 16-byte piece of a contiguous 512-byte row.
    //   whole tile:  stg != NULL; tokens t_base + tg + TG j below t_lim (one staged chunk of tokens)
    //   split tile:  stg == NULL; tokens my + n (tg + TG j): contributor `my` of n takes the tokens t = my (mod n)
    //                and adds the partials up in ascending K order; it first waits (bounded) until all n have
    //                published, and fetches what the epilogue itself reads (residual stream, rotary table) for its
    //                first tokens before that wait.
    // Returns false when the wait gave up.
    auto others_there = [&](int tile, int n, int gi, int grp, int G) -> bool {
      if (gi == 0) {
        wait_flag[4 + grp] = counter_wait(p.counters + tile, (p.gen << 8) + n, p.status, p.wait_limit) && !*abort_flag;
        TRACE(6);
      }
      // The polling thread's acquire and the barrier order the others' reads of the partial sums behind the
      // contributors' releases; those reads go to L2 (ld.global.cg), so no fence of their own is needed.
      if (G == 128) epi_barrier(); else group_barrier(grp);
      if (gi == 0 && grp == 0) TRACE(9);
      return wait_flag[4 + grp] != 0;
    };

    auto finish_plain = [&](int tile, int gi, int G, int grp, int my, int n, int first, const float *stg, int t_base,
                            int t_lim) -> bool {
      int seg, row0, col0, valid;
      locate(p, tile, seg, row0, col0, valid);
      const int ng = gi & 31, tg = gi >> 5, TG = G >> 5;
      const int col = col0 + 4 * ng;
      // Every matrix has a multiple of 8 output features (the shape checks see to it), so a thread's four columns are
      // inside the matrix together or not at all.
      const bool full4 = 4 * ng < valid;
      const int js = n * TG;                                         // token step inside a batch of four
      const int cm = row0 + 4 * ng;                                  // first of this thread's 4 columns inside q, k or v
      const int half = p.head_dim >> 1;
      const bool upper = (cm & half) != 0;
      const bool res_norm = p.mode == MODE_RESIDUAL && p.gain != nullptr;
      const bool rope = p.mode == MODE_QKV && seg != 2;
      float gn[4] = {0.f, 0.f, 0.f, 0.f};
      if (res_norm) {
#pragma unroll
        for (int e = 0; e < 4; ++e) gn[e] = full4 ? __bfloat162float(p.gain[col + e]) : 0.f;
      }
      // what the epilogue reads besides the accumulators, for the four tokens of a batch at once
      auto load_ops = [&](int tb, float4 *oa, float4 *ob) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int t = tb + j * js;
          oa[j] = ob[j] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (t >= t_lim) continue;
          if (res_norm) {
            const float *y = p.out_f32 + (size_t)t * p.ldo + col;
            if (full4) oa[j] = *reinterpret_cast<const float4 *>(y);
          } else if (rope) {
            const size_t ti = (size_t)spos[t] * half + (cm & (half - 1));
            oa[j] = *reinterpret_cast<const float4 *>(p.cos_t + ti);
            ob[j] = *reinterpret_cast<const float4 *>(p.sin_t + ti);
          }
        }
      };
      const int tb0 = t_base + my + n * tg;
      float4 oa[4], ob[4];
      if (tb0 < t_lim) load_ops(tb0, oa, ob);
      if (!stg && !others_there(tile, n, gi, grp, G)) return false;
      for (int tb = tb0; tb < t_lim; tb += 4 * js) {                 // tokens are uniform inside a warp
        if (tb != tb0) load_ops(tb, oa, ob);
        float4 acc[4];
        if (stg) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int t = tb + j * js;
            acc[j] = t < t_lim ? *reinterpret_cast<const float4 *>(stg + (size_t)(t - t_base) * STAGE_PITCH + 4 * ng)
                               : make_float4(0.f, 0.f, 0.f, 0.f);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
          for (int c0 = 0; c0 < n; c0 += 4) {
            float4 tmp[4][4];
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
              const int owner = first + c0 + cc;
              const float *src = p.scratch + ((size_t)owner * 2 + w.owner_slot(tile, owner)) * SLOT_FLOATS + 4 * ng;
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int t = tb + j * js;
                tmp[cc][j] = (c0 + cc < n && t < t_lim) ? __ldcg((const float4 *)(src + (size_t)t * TILE_N))
                                                         : make_float4(0.f, 0.f, 0.f, 0.f);
              }
            }
#pragma unroll
            for (int cc = 0; cc < 4; ++cc)
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                acc[j].x += tmp[cc][j].x; acc[j].y += tmp[cc][j].y; acc[j].z += tmp[cc][j].z; acc[j].w += tmp[cc][j].w;
              }
          }
        }
        if (!stg && tb == tb0 && gi == 0 && grp == 0) {
          if (acc[0].x == 1.2345e-30f) TRACE(14);                    // (keeps the partial sums live up to here)
          TRACE(12);
        }
        if (res_norm) {
          // new residual stream, its bf16(gain * x) image for the next GEMM, and this tile's sums of squares
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int t = tb + j * js;
            if (t >= t_lim) continue;                                // uniform inside the warp
            float *y = p.out_f32 + (size_t)t * p.ldo + col;
            const float yn[4] = {oa[j].x + acc[j].x, oa[j].y + acc[j].y, oa[j].z + acc[j].z, oa[j].w + acc[j].w};
            float sq = 0.f;
#pragma unroll
            for (int e = 0; e < 4; ++e)
              if (full4) sq += yn[e] * yn[e];
            if (full4) {
              *reinterpret_cast<float4 *>(y) = make_float4(yn[0], yn[1], yn[2], yn[3]);
              __nv_bfloat162 lo = __floats2bfloat162_rn(gn[0] * yn[0], gn[1] * yn[1]);
              __nv_bfloat162 hi = __floats2bfloat162_rn(gn[2] * yn[2], gn[3] * yn[3]);
              *reinterpret_cast<uint2 *>(p.xb + (size_t)t * p.ldo + col) = make_uint2(*(uint32_t *)&lo, *(uint32_t *)&hi);
            }
#pragma unroll
            for (int o = 16; o; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
            if (lane == 0) p.ss_out[(size_t)tile * OURO_MAX_ROWS + t] = sq;
          }
          continue;
        }
        if (p.mode == MODE_QKV) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int t = tb + j * js;
            if (t >= t_lim) continue;                                // uniform inside the warp
            const float r = rs[t];
            const float vals[4] = {acc[j].x * r, acc[j].y * r, acc[j].z * r, acc[j].w * r};
            float other[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) other[e] = __shfl_xor_sync(0xffffffffu, vals[e], half >> 2);
            const float cs[4] = {oa[j].x, oa[j].y, oa[j].z, oa[j].w}, sn[4] = {ob[j].x, ob[j].y, ob[j].z, ob[j].w};
            float rv[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
              rv[e] = seg == 2 ? vals[e] : (upper ? vals[e] * cs[e] + other[e] * sn[e] : vals[e] * cs[e] - other[e] * sn[e]);
            __nv_bfloat16 *dst = seg == 0 ? p.q_out + (size_t)t * p.dq + cm
                               : seg == 1 ? p.k_out + (size_t)(p.L + t) * p.dkv + cm
                                          : p.v_out + (size_t)(p.L + t) * p.dkv + cm;
            if (full4) {
              __nv_bfloat162 lo = __floats2bfloat162_rn(rv[0], rv[1]), hi = __floats2bfloat162_rn(rv[2], rv[3]);
              *reinterpret_cast<uint2 *>(dst) = make_uint2(*(uint32_t *)&lo, *(uint32_t *)&hi);
            }
          }
          continue;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int t = tb + j * js;
          if (t >= t_lim) continue;                                  // uniform inside the warp
          const float r = rs[t];
          const float vals[4] = {acc[j].x * r, acc[j].y * r, acc[j].z * r, acc[j].w * r};
          if (p.mode == MODE_HEAD && !stg) {                         // the warp's 32 lanes hold the tile's 128 columns
            uint32_t bu = 0;
            int bi = col;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              uint32_t uo = ordered_u32(vals[e]);
              if (full4 && uo > bu) { bu = uo; bi = col + e; }
            }
            const uint32_t mx = __reduce_max_sync(0xffffffffu, bu);
            const int src_lane = __ffs(__ballot_sync(0xffffffffu, bu == mx)) - 1;   // lowest lane = smallest index
            bi = __shfl_sync(0xffffffffu, bi, src_lane);
            if (lane == 0) {
              p.tile_max[(size_t)tile * OURO_MAX_ROWS + t] = ordered_f32(mx);
              p.tile_arg[(size_t)tile * OURO_MAX_ROWS + t] = bi;
            }
          }
          if (p.out_f32) {
            float *y = p.out_f32 + (size_t)t * p.ldo + col;
            const bool add = p.mode == MODE_RESIDUAL;
            if (full4) {                                              // the row pitch is a multiple of 4 as well
              float4 o4 = make_float4(vals[0], vals[1], vals[2], vals[3]);
              if (add) { const float4 y4 = *reinterpret_cast<const float4 *>(y); o4.x += y4.x; o4.y += y4.y; o4.z += y4.z; o4.w += y4.w; }
              *reinterpret_cast<float4 *>(y) = o4;
            }
          }
        }
      }
      return true;
    };

    // SiLU(gate) * up: a tile holds 64 output features, gate in tile rows 0..63 and up in rows 64..127
    auto finish_swiglu = [&](int tile, int gi, int G, int grp, int my, int n, int first, const float *stg, int t_base,
                             int t_lim) -> bool {
      const int F = p.a_rows[0];
      const int ng = gi & 15, tg = gi >> 4, TG = G >> 4;             // 4 features; tokens my + n (tg + TG j)
      const int feat = tile * 64 + 4 * ng;
      const int js = n * TG;
      if (!stg && !others_there(tile, n, gi, grp, G)) return false;
      for (int tb = t_base + my + n * tg; tb < t_lim; tb += 4 * js) {
        float4 g[4], u[4];
        if (stg) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int t = tb + j * js;
            g[j] = u[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (t < t_lim) {
              g[j] = *reinterpret_cast<const float4 *>(stg + (size_t)(t - t_base) * STAGE_PITCH + 4 * ng);
              u[j] = *reinterpret_cast<const float4 *>(stg + (size_t)(t - t_base) * STAGE_PITCH + 64 + 4 * ng);
            }
          }
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) g[j] = u[j] = make_float4(0.f, 0.f, 0.f, 0.f);
          for (int c0 = 0; c0 < n; c0 += 4) {
            float4 tg4[4][4], tu4[4][4];
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
              const int owner = first + c0 + cc;
              const float *src = p.scratch + ((size_t)owner * 2 + w.owner_slot(tile, owner)) * SLOT_FLOATS + 4 * ng;
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int t = tb + j * js;
                const bool in = c0 + cc < n && t < t_lim;
                tg4[cc][j] = in ? __ldcg((const float4 *)(src + (size_t)t * TILE_N)) : make_float4(0.f, 0.f, 0.f, 0.f);
                tu4[cc][j] = in ? __ldcg((const float4 *)(src + (size_t)t * TILE_N + 64)) : make_float4(0.f, 0.f, 0.f, 0.f);
              }
            }
#pragma unroll
            for (int cc = 0; cc < 4; ++cc)
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                g[j].x += tg4[cc][j].x; g[j].y += tg4[cc][j].y; g[j].z += tg4[cc][j].z; g[j].w += tg4[cc][j].w;
                u[j].x += tu4[cc][j].x; u[j].y += tu4[cc][j].y; u[j].z += tu4[cc][j].z; u[j].w += tu4[cc][j].w;
              }
          }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int t = tb + j * js;
          if (t < t_lim && feat < F) {
            const float r = rs[t];
            g[j].x *= r; g[j].y *= r; g[j].z *= r; g[j].w *= r;
            u[j].x *= r; u[j].y *= r; u[j].z *= r; u[j].w *= r;
            __nv_bfloat162 lo = __floats2bfloat162_rn(silu(g[j].x) * u[j].x, silu(g[j].y) * u[j].y);
            __nv_bfloat162 hi = __floats2bfloat162_rn(silu(g[j].z) * u[j].z, silu(g[j].w) * u[j].w);
            *(uint2 *)(p.out_bf16 + (size_t)t * F + feat) = make_uint2(*(uint32_t *)&lo, *(uint32_t *)&hi);
          }
        }
      }
      return true;
    };

    // Partial tiles.  Called once this CTA has published all its own partials, so waiting for the others cannot
    // form a cycle.  The (at most two) tiles are finished side by side, each by one half of the epilogue threads.
    auto run_fixups = [&]() {
      const int grp = et >> 6, gi = et & 63;
      bool mine = true;
      if (grp < n_pend) {
        const int tile = pend_tile[grp], n = pend_n[grp], first = pend_first[grp], my = (int)blockIdx.x - first;
        mine = p.mode == MODE_SWIGLU ? finish_swiglu(tile, gi, 64, grp, my, n, first, nullptr, 0, rows)
                                     : finish_plain(tile, gi, 64, grp, my, n, first, nullptr, 0, rows);
        if (gi == 0 && grp == 0) TRACE(10);
        if (mine) {
          if (publish) __threadfence();                                // this thread's outputs, before the tile counts as finished
          group_barrier(grp);
          // every contributor counts towards the hand-over itself: the GEMM is finished once all shares of all tiles
          // are (the host passes the total), and nobody has to learn that it was the last of its tile
          if (gi == 0 && publish) atomicAdd(cp.finished + ci, 1);
        }
      }
      if (gi == 0 && grp == 0) TRACE(11);
      if (!mine) wait_flag[2] = 1;
      epi_barrier();
      if (wait_flag[2]) ok = false;
      n_pend = 0;
    };

    if (ci > 0) {
      // this GEMM's per-token factors are sums over all tiles of the GEMM before it
      if (et == 0) wait_flag[0] = chain_wait(cp, ci - 1) && !*abort_flag;
      epi_barrier();
      ok = wait_flag[0] != 0;
      epi_barrier();
      if (!ok) break;
      __threadfence();
    }
    if (et < OURO_MAX_ROWS) {
      float r = 1.0f;
      if (p.ss_in && et < rows) {
        float sum = 0.f;
        for (int i = 0; i < p.ss_tiles; ++i) sum += p.ss_in[(size_t)i * OURO_MAX_ROWS + et];
        r = 1.0f / sqrtf(sum * p.ss_inv_d + p.eps);
      }
      rs[et] = r;
      spos[et] = (p.mode == MODE_QKV && et < rows) ? p.pos[et] : 0;
    }
    if (et == 0) wait_flag[2] = 0;
    epi_barrier();

    while (w.next(s)) {
      int a = item & 1;
      // the stream-K spans come first: once the whole tiles start, this CTA has published all its partials and
      // can add up its shares while the tensor cores work on the whole tile
      if (s.n_contrib == 1 && n_pend > 0) run_fixups();
      if (!ok) break;
      // one thread waits (bounded) and tells the others, so that all 128 leave the loop together
      if (et == 0) wait_flag[a] = mbar_wait(&acc_full[a], (item >> 1) & 1, abort_flag) && !*abort_flag;
      epi_barrier();
      ok = wait_flag[a] != 0;
      if (!ok) break;
      if (et == 0) TRACE(4);                       // overwritten per item: the last accumulator's arrival remains
      fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * acc_cols;
      if (s.n_contrib == 1) {
        // whole tile: the accumulators go to shared memory token-major, STAGE_TOK tokens at a time, and are finished
        // from there; the TMEM buffer is handed back as soon as it has been read
        for (int c0 = 0; c0 < p.t_pad; c0 += STAGE_TOK) {
          const int c1 = min(p.t_pad, c0 + STAGE_TOK);
          for (int t0 = c0; t0 < c1; t0 += 16) {
            tmem_ld16(taddr + t0, v);
#pragma unroll
            for (int i = 0; i < 16; ++i) stage[(t0 - c0 + i) * STAGE_PITCH + nl] = v[i];
          }
          if (c1 == p.t_pad) {
            fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[a]);
          }
          epi_barrier();
          const int lim = min(c1, rows);
          if (p.mode == MODE_SWIGLU) {
            finish_swiglu(s.tile, et, 128, 0, 0, 1, 0, stage, c0, lim);
          } else if (p.mode == MODE_HEAD) {
            // greedy choice inside the tile: two threads per token scan 64 parked logits each in ascending index
            // order (a strict comparison keeps the smallest index among equals), then the halves are compared
            int seg, row0, col0, valid;
            locate(p, s.tile, seg, row0, col0, valid);
            const int t = c0 + (et >> 1), h = et & 1;
            uint32_t bu = 0;
            int bi = col0 + 64 * h;
            if (t < lim) {
              const float r = rs[t];
              const float *row = stage + (size_t)(t - c0) * STAGE_PITCH + 64 * h;
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                const float4 x4 = *reinterpret_cast<const float4 *>(row + 4 * i);
                const float xs[4] = {x4.x * r, x4.y * r, x4.z * r, x4.w * r};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const int cidx = 64 * h + 4 * i + e;
                  const uint32_t uo = ordered_u32(xs[e]);
                  if (cidx < valid && uo > bu) { bu = uo; bi = col0 + cidx; }
                }
              }
            }
            const uint32_t ou = __shfl_xor_sync(0xffffffffu, bu, 1);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, 1);
            if (ou > bu || (ou == bu && oi < bi)) { bu = ou; bi = oi; }
            if (t < lim && h == 0) {
              p.tile_max[(size_t)s.tile * OURO_MAX_ROWS + t] = ordered_f32(bu);
              p.tile_arg[(size_t)s.tile * OURO_MAX_ROWS + t] = bi;
            }
          }
          // one call site for every other mode (the routine is inlined: a second site would be a second copy of it)
          if (p.mode != MODE_SWIGLU && (p.mode != MODE_HEAD || p.out_f32)) finish_plain(s.tile, et, 128, 0, 0, 1, 0, stage, c0, lim);
          if (publish && c1 == p.t_pad) __threadfence();
          epi_barrier();
          if (publish && c1 == p.t_pad && et == 0) atomicAdd(cp.finished + ci, 1);
        }
      } else {
        // partial tile: park it in this CTA's slot and announce it; the partials are added up after the loop
        float *mine = p.scratch + ((size_t)blockIdx.x * 2 + s.slot) * SLOT_FLOATS;
        for (int t0 = 0; t0 < p.t_pad; t0 += 16) {
          tmem_ld16(taddr + t0, v);
#pragma unroll
          for (int i = 0; i < 16; ++i)
            if (t0 + i < rows) __stcg(mine + (size_t)(t0 + i) * TILE_N + nl, v[i]);
        }
        fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[a]);
        __threadfence();
        epi_barrier();
        if (et == 0) {                             // first of this generation to get here: replaces what an earlier GEMM left
          atomicMax(p.counters + s.tile, p.gen << 8);
          atomicAdd(p.counters + s.tile, 1);
        }
        pend_tile[n_pend] = s.tile;
        pend_n[n_pend] = s.n_contrib;
        pend_first[n_pend] = s.first_owner;
        ++n_pend;
      }
      ++item;
    }
    if (et == 0) TRACE(5);
    if (ok) run_fixups();
    if (et == 0) TRACE(7);
    }
    if (!ok && et == 0) { *abort_flag = 1; atomicExch(p0.status, 1); }
  }
  // ------------------------------------------------------------------ teardown
  fence_before_sync();
  __syncthreads();
  if (*abort_flag && ((warp == 0 && lane < W_PRODUCERS) || (warp == 6 && lane == 0))) {
    // Somebody gave up: copies this lane issued may still be landing in this CTA's shared memory.  Wait (bounded) for
    // the last one of every stage before the CTA leaves; a stage whose other half was never requested cannot
    // complete its phase, which the limit covers (the bytes themselves arrive within microseconds).
    for (int st = 0; st < n_stages; ++st) {
      if (n_issued <= (uint32_t)st) continue;
      const uint32_t last = ((n_issued - 1 - st) / n_stages) * n_stages + st;      // last copy issued into this stage
      mbar_wait(&full[st], (last / n_stages) & 1, nullptr, 1u << 14);
    }
  }
  if (*abort_flag && warp == 1 && lane == 0) {     // ... and no contraction may still be running when TMEM is given back
    mma_commit(drain_bar);
    mbar_wait(drain_bar, 0, nullptr, 1u << 16);
  }
  __syncthreads();
  if (warp == 1) {
    fence_after_sync();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)(2 * acc_cols)));
  }
}

// ------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

bool make_map(CUtensorMap *m, const void *base, int rows, int K, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {BLOCK_K, (cuuint32_t)box_rows};
  cuuint32_t es[2] = {1, 1};
  return g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct LayerMaps {
  CUtensorMap wq, wk, wv, wo, wg, wu, wd;
};
struct FastModel {
  bool ok = false;
  std::vector<LayerMaps> layers;
  CUtensorMap head;
  CUtensorMap kmap, vmap;               // K and V caches as [layers * max_seq][kv width], box 64 x 128 (tcgen05 attention)
  bool kv_maps = false;
  CUtensorMap x_d[8], x_q[8], x_f[8];   // activations normed [128, d], attention out [128, dq], SwiGLU out [128, F]; box rows 16, 32, .., 128
};
struct FastState {
  FastModel m[2];
  int grid = 0;
  int smem_max = 0;
  float *slots = nullptr;
  int *counters = nullptr;
  float *attn_part = nullptr;   // per-chunk softmax pieces of the split attention
  float *tile_max = nullptr;    // LM head: per-tile best logit and index of every token
  int *tile_arg = nullptr;
  float *ss = nullptr;          // per-tile sums of squares of the residual stream (RMSNorm folded into the GEMMs)
  int *finished = nullptr;      // [MAX_CHAIN] finished-tile counters of the chained GEMMs (device)
  int finished_host[MAX_CHAIN + 1] = {0, 0, 0, 0, 0};   // the values those counters have once everything launched so far is done
  ChainParams chain{};          // GEMMs collected for the next launch
  int chain_kind[MAX_CHAIN] = {0, 0, 0, 0};
  bool fuse = true;             // run consecutive GEMMs as one launch
  long pf_ffn_rows = 0;         // rows of gate and of up the attention kernel prefetches into L2 besides the output projection (< 0: nothing)
  int gen_next = 1;             // generation number of the next GEMM (tile counters carry it, see GemmParams::counters)
  bool dirty = false;           // a bounded wait gave up: counters must be cleared before the next launch
  uint32_t wait_limit = 1u << 22;   // polls of a partial-tile wait (ouro_debug_set_wait_limit)
};
constexpr int MAX_TILES = 4096;
constexpr int SPARE_BYTES = 2048;          // behind the tile counters: chain counters [0, 64), attention arrival counters [64, 512)

size_t slots_bytes() { return (size_t)MAX_GRID * 2 * SLOT_FLOATS * sizeof(float); }
size_t tile_best_bytes() { return (size_t)MAX_TILES * OURO_MAX_ROWS * 4; }
constexpr int MAX_SS_TILES = 64;           // d_model <= 8192
size_t ss_bytes() { return (size_t)MAX_SS_TILES * OURO_MAX_ROWS * sizeof(float); }

int stages_for(int t_pad, int smem_max) {
  int stage = A_BYTES + t_pad * BLOCK_K * 2;
  int fixed = 1024 + STAGE_BYTES + 1536;  // alignment slack, parked whole tile, barriers, flags, per-token factors and positions
  int s = (smem_max - fixed) / stage;
  return s > 12 ? 12 : s;
}

}  // namespace

struct ouro_fast { FastState s; };

size_t ouro_scratch_bytes(const ouro_model_desc *t, const ouro_model_desc *d) {
  size_t attn = attention_tc_scratch_bytes(*t);
  if (d && attention_tc_scratch_bytes(*d) > attn) attn = attention_tc_scratch_bytes(*d);
  return slots_bytes() + 2 * MAX_TILES * sizeof(int) + SPARE_BYTES + 2 * tile_best_bytes() + ss_bytes() + attn;
}

static bool shape_ok(const ouro_model_desc &d) {
  int dq = d.n_heads * d.head_dim;
  return d.dtype == OURO_BF16 && d.d_model % 64 == 0 && d.d_model <= MAX_SS_TILES * TILE_N && dq % 64 == 0 && d.d_ffn % 64 == 0 && d.vocab % 8 == 0 &&
         (d.vocab + TILE_N - 1) / TILE_N <= MAX_TILES && (2 * d.d_ffn + TILE_N - 1) / TILE_N <= MAX_TILES;
}

int ouro_fast_setup(ouro_ctx *c) {
  c->fast = nullptr;
  bool any = false;
  for (auto &M : c->m) any = any || (M.present && shape_ok(M.d));
  if (!any) return OURO_OK;
  int dev = 0, sms = 0, smem = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
    c->err = "device attributes unavailable";
    return OURO_ECUDA;
  }
  if (!g_encode) {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn) {
      c->err = "cuTensorMapEncodeTiled unavailable";
      return OURO_ECUDA;
    }
    g_encode = (EncodeTiledFn)fn;
  }
  ouro_fast *f = new ouro_fast();
  f->s.grid = sms < MAX_GRID ? sms : MAX_GRID;
  f->s.smem_max = smem;
  f->s.slots = c->a.scratch;
  f->s.counters = (int *)((char *)c->a.scratch + slots_bytes());
  f->s.finished = f->s.counters + 2 * MAX_TILES;               // inside the spare words behind the tile counters
  {
    const char *e = getenv("OURO_FUSE");                       // OURO_FUSE=0: every GEMM is a launch of its own
    f->s.fuse = !(e && e[0] == '0');
    const char *pf = getenv("OURO_PF_ROWS");
    if (pf) f->s.pf_ffn_rows = atol(pf);
    const char *g0 = getenv("OURO_GEN_START");                  // test aid: first generation number of the tile counters
    if (g0 && atoi(g0) > 0 && atoi(g0) < (1 << 22)) f->s.gen_next = atoi(g0);
  }
  f->s.tile_max = (float *)((char *)c->a.scratch + slots_bytes() + 2 * MAX_TILES * sizeof(int) + SPARE_BYTES);
  f->s.tile_arg = (int *)((char *)f->s.tile_max + tile_best_bytes());
  f->s.ss = (float *)((char *)f->s.tile_arg + tile_best_bytes());
  f->s.attn_part = (float *)((char *)f->s.ss + ss_bytes());
  if (cudaMemsetAsync(f->s.counters, 0, 2 * MAX_TILES * sizeof(int) + SPARE_BYTES, c->stream) != cudaSuccess ||
      cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
      attention_tc_setup() != OURO_OK || attention_tm_setup() != OURO_OK) {
    delete f;
    c->err = "tensor-core GEMM set-up failed";
    return OURO_ECUDA;
  }
  for (int w = 0; w < 2; ++w) {
    ModelRt &M = c->m[w];
    if (!M.present || !shape_ok(M.d)) continue;
    const ouro_model_desc &d = M.d;
    FastModel &fm = f->s.m[w];
    const int dq = d.n_heads * d.head_dim, dkv = d.n_kv_heads * d.head_dim;
    bool ok = true;
    fm.layers.resize(d.n_layers);
    for (int l = 0; l < d.n_layers && ok; ++l) {
      LayerMaps &lm = fm.layers[l];
      ok = make_map(&lm.wq, M.wq[l], dq, d.d_model, TILE_N) && make_map(&lm.wk, M.wk[l], dkv, d.d_model, TILE_N) &&
           make_map(&lm.wv, M.wv[l], dkv, d.d_model, TILE_N) && make_map(&lm.wo, M.wo[l], d.d_model, dq, TILE_N) &&
           make_map(&lm.wg, M.w_gate[l], d.d_ffn, d.d_model, 64) && make_map(&lm.wu, M.w_up[l], d.d_ffn, d.d_model, 64) &&
           make_map(&lm.wd, M.w_down[l], d.d_model, d.d_ffn, TILE_N);
    }
    ok = ok && make_map(&fm.head, M.lm_head, d.vocab, d.d_model, TILE_N);
    if (ok && attention_tm_supported(d)) {
      ok = make_map(&fm.kmap, M.k_cache, d.n_layers * d.max_seq, dkv, 128) && make_map(&fm.vmap, M.v_cache, d.n_layers * d.max_seq, dkv, 128);
      fm.kv_maps = ok;
    }
    for (int i = 0; i < 8 && ok; ++i)
      ok = make_map(&fm.x_d[i], c->a.xn, OURO_MAX_ROWS, d.d_model, 16 * (i + 1)) &&
           make_map(&fm.x_q[i], c->a.att, OURO_MAX_ROWS, dq, 16 * (i + 1)) &&
           make_map(&fm.x_f[i], c->a.act, OURO_MAX_ROWS, d.d_ffn, 16 * (i + 1));
    if (!ok) {
      delete f;
      c->err = "cuTensorMapEncodeTiled failed";
      return OURO_ECUDA;
    }
    fm.ok = true;
  }
  c->fast = f;
  return OURO_OK;
}

void ouro_fast_teardown(ouro_ctx *c) {
  delete c->fast;
  c->fast = nullptr;
}

// The weight side of one GEMM of the forward: which matrices, how they are tiled, how long K is.
enum { G_QKV = 0, G_WO = 1, G_GATEUP = 2, G_DOWN = 3, G_HEAD = 4 };
struct WeightSide {
  CUtensorMap a[3];
  int a_tiles[3] = {0, 0, 0}, a_rows[3] = {0, 0, 0}, a_count = 1, tiles = 0, K = 0;
  bool swiglu = false;
};
static WeightSide weight_side(const ouro_model_desc &d, const FastModel &fm, int l, int kind) {
  auto tiles = [](int n) { return (n + TILE_N - 1) / TILE_N; };
  const int dq = d.n_heads * d.head_dim, dkv = d.n_kv_heads * d.head_dim;
  WeightSide w;
  switch (kind) {
    case G_QKV: {
      const LayerMaps &lm = fm.layers[l];
      w.a[0] = lm.wq; w.a[1] = lm.wk; w.a[2] = lm.wv;
      w.a_tiles[0] = tiles(dq); w.a_tiles[1] = tiles(dkv); w.a_tiles[2] = tiles(dkv);
      w.a_rows[0] = dq; w.a_rows[1] = dkv; w.a_rows[2] = dkv;
      w.a_count = 3;
      w.tiles = w.a_tiles[0] + w.a_tiles[1] + w.a_tiles[2];
      w.K = d.d_model;
      break;
    }
    case G_WO:
      w.a[0] = fm.layers[l].wo; w.a_tiles[0] = tiles(d.d_model); w.a_rows[0] = d.d_model;
      w.tiles = w.a_tiles[0];
      w.K = dq;
      break;
    case G_GATEUP:
      w.a[0] = fm.layers[l].wg; w.a[1] = fm.layers[l].wu; w.a_rows[0] = d.d_ffn; w.a_count = 2;
      w.tiles = (d.d_ffn + 63) / 64;
      w.K = d.d_model;
      w.swiglu = true;
      break;
    case G_DOWN:
      w.a[0] = fm.layers[l].wd; w.a_tiles[0] = tiles(d.d_model); w.a_rows[0] = d.d_model;
      w.tiles = w.a_tiles[0];
      w.K = d.d_ffn;
      break;
    default:
      w.a[0] = fm.head; w.a_tiles[0] = tiles(d.vocab); w.a_rows[0] = d.vocab;
      w.tiles = w.a_tiles[0];
      w.K = d.d_model;
      break;
  }
  return w;
}
static void set_weights(GemmParams &p, const WeightSide &w) {
  for (int i = 0; i < 3; ++i) { p.a[i] = w.a[i]; p.a_tiles[i] = w.a_tiles[i]; p.a_rows[i] = w.a_rows[i]; }
  p.a_count = w.a_count;
  p.tiles = w.tiles;
}
static int grid_for(const FastState &s, int tiles, int kb) {
  const long total = (long)tiles * kb;
  return total < s.grid ? (int)total : s.grid;
}
// What the hand-over counter of a GEMM reaches: one count per whole tile and one per contributor of a split tile
// (the schedule of weight_stream.cuh, worked out on the host).
static int finish_units(int tiles, int kb, int grid) {
  const int t0 = (tiles / grid) * grid, rem = tiles - t0;
  if (rem == 0) return tiles;
  const int total = rem * kb, per = (total + grid - 1) / grid;
  int units = t0;
  for (int rel = 0; rel < rem; ++rel) units += (rel * kb + kb - 1) / per - (rel * kb) / per + 1;
  return units;
}
// Launches the GEMMs collected so far as one chain.
static void flush_chain(ouro_ctx *c) {
  FastState &s = c->fast->s;
  ChainParams &cp = s.chain;
  if (cp.n == 0) return;
  OURO_COUNT_LAUNCH();
  int grid = 1;
  for (int i = 0; i < cp.n; ++i) grid = std::max(grid, grid_for(s, cp.g[i].tiles, cp.g[i].kb));
  cp.finished = s.finished;
  if (s.gen_next + MAX_CHAIN >= (1 << 22)) {                 // generation numbers used up: start over on cleared words
    cudaMemsetAsync(s.counters, 0, MAX_TILES * sizeof(int), c->stream);
    s.gen_next = 1;
  }
  for (int i = 0; i < cp.n; ++i) cp.g[i].gen = s.gen_next++;
  for (int i = 0; i + 1 < cp.n; ++i) cp.target[i] = (s.finished_host[i] += finish_units(cp.g[i].tiles, cp.g[i].kb, grid));
  if (cp.fold.part || cp.embed.table) cp.fold_target = (s.finished_host[MAX_CHAIN] += grid);
  const bool per_kind = cp.n == 1 && c->prof_class >= OURO_PROF_QKV && c->prof_class <= OURO_PROF_HEAD;
  static const int kind_class[5] = {OURO_PROF_QKV, OURO_PROF_WO, OURO_PROF_GATEUP, OURO_PROF_DOWN, OURO_PROF_HEAD};
  {
    ProfScope ps(c, per_kind ? kind_class[s.chain_kind[0]] : OURO_PROF_GEMM);
    launch_pdl(gemm_tc_kernel, grid, THREADS, (size_t)s.smem_max, c->stream, cp);
  }
  cp.n = 0;
  cp.fold.part = nullptr;
  cp.embed.table = nullptr;
}

// Adds a GEMM to the chain under construction; `last` launches the chain (something other than a GEMM follows).
static void push_gemm(ouro_ctx *c, GemmParams &p, int kind, const CUtensorMap *xmaps, int K, int rows, bool last) {
  FastState &s = c->fast->s;
  p.kb = K / BLOCK_K;
  p.rows = rows;
  p.t_pad = (rows + 15) & ~15;
  p.b = xmaps[p.t_pad / 16 - 1];
  p.stages = stages_for(p.t_pad, s.smem_max);
  p.scratch = s.slots;
  p.counters = s.counters;
  p.status = &c->st->status;
  p.rows_dev = c->cur_rows_dev;
  p.trace_id = kind;
  p.wait_limit = s.wait_limit;
  if (s.chain.n > 0 && s.chain.g[0].rows != rows) flush_chain(c);   // cannot happen inside one forward
  s.chain_kind[s.chain.n] = kind;
  s.chain.g[s.chain.n++] = p;
  // one launch per GEMM when asked for, and while a single kind of GEMM is being timed
  const bool split = !s.fuse || (c->prof_class >= OURO_PROF_QKV && c->prof_class <= OURO_PROF_HEAD);
  if (last || split || s.chain.n == MAX_CHAIN) flush_chain(c);
}

// Clears what an aborted launch may have left behind (tile counters, chain counters).
void ouro_fast_reset(ouro_ctx *c, bool force) {
  if (!c->fast) return;
  FastState &s = c->fast->s;
  s.chain.n = 0;
  s.chain.fold.part = nullptr;
  s.chain.embed.table = nullptr;
  if (!force && !s.dirty) return;
  cudaMemsetAsync(s.counters, 0, 2 * MAX_TILES * sizeof(int) + SPARE_BYTES, c->stream);
  for (int &v : s.finished_host) v = 0;
  s.gen_next = 1;
  s.dirty = false;
}
void ouro_fast_mark_dirty(ouro_ctx *c) {
  if (c->fast) c->fast->s.dirty = true;
}
extern "C" int ouro_debug_set_wait_limit(ouro_ctx *c, int64_t polls) {
  if (!c) return OURO_EINVAL;
  if (!c->fast) return OURO_ESTATE;
  c->fast->s.wait_limit = polls < 0 ? (1u << 22) : (uint32_t)std::min<int64_t>(polls, 1u << 22);
  return OURO_OK;
}

// The row count of a candidate block may stay on the device when every kernel of the forward reads it from there:
// the tensor-core GEMMs with the rotary epilogue and one of the two tensor-core attention kernels.
bool ouro_fast_available(ouro_ctx *c, int which) {
  if (!c->fast || !c->fast->s.m[which].ok) return false;
  const ouro_model_desc &d = c->m[which].d;
  return d.head_dim == 64 || d.head_dim == 128;
}

// The embedding gather runs in front of the first layer's q,k,v GEMM, inside its launch.
int ouro_fast_embed(ouro_ctx *c, int which, int rows) {
  if (!c->fast || !c->fast->s.m[which].ok) return OURO_ESTATE;
  ModelRt &M = c->m[which];
  ChainParams &cp = c->fast->s.chain;
  cp.n = 0;
  cp.fold.part = nullptr;
  ChainParams::Embed &e = cp.embed;
  e.table = (const __nv_bfloat16 *)M.embed;
  e.tok = M.blk.tok;
  e.gain = (const __nv_bfloat16 *)M.attn_norm[0];
  e.x = c->a.x;
  e.xb = (__nv_bfloat16 *)c->a.xn;
  e.ss = c->fast->s.ss;
  e.rows_dev = c->cur_rows_dev;
  e.rows = rows;
  e.d = M.d.d_model;
  return OURO_OK;
}

// One decoder layer with the tensor-core GEMMs; OURO_ESTATE when the model does not qualify.
int ouro_fast_layer(ouro_ctx *c, int which, int l, int rows) {
  if (!c->fast || !c->fast->s.m[which].ok) return OURO_ESTATE;
  ModelRt &M = c->m[which];
  FastModel &fm = c->fast->s.m[which];
  const ouro_model_desc &d = M.d;
  const int dq = d.n_heads * d.head_dim, dkv = d.n_kv_heads * d.head_dim;
  Activations &a = c->a;
  cudaStream_t s = c->stream;
  auto tiles = [](int n) { return (n + TILE_N - 1) / TILE_N; };
  // a.xn holds bf16(attn_norm * x) and ss the sums of squares, left by the embedding or the previous layer's down GEMM
  float *ss = c->fast->s.ss;
  const int ss_tiles = tiles(d.d_model);
  auto consume = [&](GemmParams &p) { p.ss_in = ss; p.ss_tiles = ss_tiles; p.ss_inv_d = 1.0f / (float)d.d_model; p.eps = d.rms_eps; };
  auto produce = [&](GemmParams &p, const void *gain) { p.gain = (const __nv_bfloat16 *)gain; p.xb = (__nv_bfloat16 *)a.xn; p.ss_out = ss; };
  {
    GemmParams p{};
    set_weights(p, weight_side(d, fm, l, G_QKV));
    consume(p);
    const bool fused_rope = d.head_dim == 64 || d.head_dim == 128;   // tiles then hold whole heads
    if (fused_rope) {
      const size_t off = (size_t)l * d.max_seq * dkv;
      p.mode = MODE_QKV;
      p.pos = M.blk.pos; p.cos_t = M.rope_cos; p.sin_t = M.rope_sin;
      p.q_out = (__nv_bfloat16 *)a.q;
      p.k_out = (__nv_bfloat16 *)M.k_cache + off;
      p.v_out = (__nv_bfloat16 *)M.v_cache + off;
      p.head_dim = d.head_dim; p.dq = dq; p.dkv = dkv; p.L = M.L;
    } else {
      p.mode = MODE_STORE;
      p.out_f32 = a.qkv;
      p.ldo = dq + 2 * dkv;
    }
    push_gemm(c, p, G_QKV, fm.x_d, d.d_model, rows, true);       // closes the chain the previous layer began
    if (!fused_rope) {
      ProfScope pr(c, OURO_PROF_ROPE);
      launch_rope_append(d, a.qkv, M.blk.pos, M.rope_cos, M.rope_sin, rows, M.L, l, a.q, M.k_cache, M.v_cache, s);
    }
  }
  {
    ProfScope ps(c, OURO_PROF_ATTENTION);
    bool pieces = false;             // the attention output is still in per-span pieces
    if (c->fast->s.m[which].kv_maps) {
      // what the launch after the attention streams first: the output projection, then the first rows of gate and up
      L2Prefetch pf;
      const size_t row_bytes = (size_t)d.d_model * 2, head = std::min<size_t>((size_t)d.d_ffn, c->fast->s.pf_ffn_rows) * row_bytes;
      if (c->fast->s.pf_ffn_rows >= 0) {
        pf.ptr[0] = M.wo[l]; pf.bytes[0] = (size_t)d.d_model * dq * 2;
        pf.ptr[1] = M.w_gate[l]; pf.bytes[1] = head;
        pf.ptr[2] = M.w_up[l]; pf.bytes[2] = head;
      }
      pieces = launch_attention_tm(d, a.q, &c->fast->s.m[which].kmap, &c->fast->s.m[which].vmap, M.k_cache, M.v_cache, M.blk, rows,
                                   M.L, M.L + rows, l, c->fast->s.attn_part, a.att, &c->st->status, c->cur_rows_dev, pf, s);
    }
    else if (attention_tc_supported(d))
      pieces = launch_attention_tc(d, a.q, M.k_cache, M.v_cache, M.blk, rows, M.L, M.L + rows, l, c->fast->s.attn_part, a.att,
                                   c->cur_rows_dev, s);
    else
      launch_attention_simple(d, a.q, M.k_cache, M.v_cache, M.blk, rows, l, a.att, s);
    if (pieces) {                    // folded by the output projection's launch, all its CTAs taking part
      fold::Params &f = c->fast->s.chain.fold;
      f.part = c->fast->s.attn_part;
      f.out = (__nv_bfloat16 *)a.att;
      f.lin_end = M.blk.lin_end;
      f.seg_len = M.blk.seg_len;
      f.rows_dev = c->cur_rows_dev;
      f.rows = rows;
      f.H = d.n_heads;
      f.cap = (d.max_seq + fold::SPAN_KEYS - 1) / fold::SPAN_KEYS;
      f.head_dim = d.head_dim;
    }
  }
  {
    GemmParams p{};
    set_weights(p, weight_side(d, fm, l, G_WO));
    p.mode = MODE_RESIDUAL;
    p.out_f32 = a.x;
    p.ldo = d.d_model;
    produce(p, M.ffn_norm[l]);
    push_gemm(c, p, G_WO, fm.x_q, dq, rows, false);
  }
  {
    GemmParams p{};
    set_weights(p, weight_side(d, fm, l, G_GATEUP));
    p.mode = MODE_SWIGLU;
    p.out_bf16 = (__nv_bfloat16 *)a.act;
    consume(p);
    push_gemm(c, p, G_GATEUP, fm.x_d, d.d_model, rows, false);
  }
  {
    GemmParams p{};
    set_weights(p, weight_side(d, fm, l, G_DOWN));
    p.mode = MODE_RESIDUAL;
    p.out_f32 = a.x;
    p.ldo = d.d_model;
    produce(p, l + 1 < d.n_layers ? M.attn_norm[l + 1] : M.final_norm);
    push_gemm(c, p, G_DOWN, fm.x_f, d.d_ffn, rows, false);     // the next layer's q,k,v or the LM head completes the chain
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    c->err = std::string("tensor-core layer launch: ") + cudaGetErrorString(e);
    return OURO_ECUDA;
  }
  return OURO_OK;
}

// Final norm, LM head and greedy choice.  The GEMM's epilogue keeps, per 128-entry vocabulary tile, each
// token's best logit and index; a small kernel then picks the best tile per token.  logits may be NULL.
__global__ void argmax_tiles_kernel(const float *tile_max, const int *tile_arg, int tiles, int32_t *out) {
  pdl_trigger();
  pdl_wait();
  const int t = blockIdx.x;
  // compared through the same order-preserving integer image as inside the tiles (-0.0 below +0.0), so that the
  // choice does not depend on where a tile boundary falls
  uint32_t bv = 0;
  int bi = INT_MAX;
  for (int i = threadIdx.x; i < tiles; i += blockDim.x) {
    uint32_t v = ordered_u32(tile_max[(size_t)i * OURO_MAX_ROWS + t]);
    int a = tile_arg[(size_t)i * OURO_MAX_ROWS + t];
    if (v > bv || (v == bv && a < bi)) { bv = v; bi = a; }
  }
  __shared__ uint32_t sv[8];
  __shared__ int si[8];
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    uint32_t ov = __shfl_xor_sync(0xffffffffu, bv, o);
    int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
  }
  if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = bv; si[threadIdx.x >> 5] = bi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w)
      if (sv[w] > bv || (sv[w] == bv && si[w] < bi)) { bv = sv[w]; bi = si[w]; }
    out[t] = bi == INT_MAX ? 0 : bi;
  }
}

int ouro_fast_head(ouro_ctx *c, int which, int rows, float *logits, int32_t *argmax_dev) {
  if (!c->fast || !c->fast->s.m[which].ok) return OURO_ESTATE;
  ModelRt &M = c->m[which];
  FastModel &fm = c->fast->s.m[which];
  const ouro_model_desc &d = M.d;
  {
    GemmParams p{};
    set_weights(p, weight_side(d, fm, 0, G_HEAD));
    p.mode = MODE_HEAD;
    p.out_f32 = logits;
    p.ldo = d.vocab;
    p.tile_max = c->fast->s.tile_max;
    p.tile_arg = c->fast->s.tile_arg;
    p.ss_in = c->fast->s.ss; p.ss_tiles = (d.d_model + TILE_N - 1) / TILE_N; p.ss_inv_d = 1.0f / (float)d.d_model; p.eps = d.rms_eps;
    push_gemm(c, p, G_HEAD, fm.x_d, d.d_model, rows, true);
  }
  {
    ProfScope ps(c, OURO_PROF_ARGMAX);
    OURO_COUNT_LAUNCH();
    launch_pdl(argmax_tiles_kernel, rows, 128, 0, c->stream, (const float *)c->fast->s.tile_max, (const int *)c->fast->s.tile_arg,
               (int)((d.vocab + TILE_N - 1) / TILE_N), argmax_dev);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    c->err = std::string("tensor-core head launch: ") + cudaGetErrorString(e);
    return OURO_ECUDA;
  }
  return OURO_OK;
}

// ===================================================================================================
// ouro_lm_head_static: the LM-head pass for callers that must not allocate.
//
// Some users of this library cannot give it a workspace: a serving process that handed all device memory to
// its own arena at start-up (a later cudaMalloc simply fails), or a latency-critical loop that must not run
// into the implicit device synchronisation an allocation can cause.  For them this one call keeps everything
// the GEMM needs besides its inputs and outputs - the partial-tile slots of the split-K schedule, the tile
// counters, the per-tile maxima and a status word - in a fixed array that is part of the library image.
// Every GPU that loads the library carries these 5 MiB until the process exits.
//
// The array's name is only meaningful in device code.  Host code must ask the runtime for its device address
// (cudaGetSymbolAddress) with the right device current; that is done once per device by the first call.
// ===================================================================================================
namespace {
constexpr int NA_GRID = 32;                        // CTAs of the static-scratch launch (slots are per CTA)
constexpr int NA_MAX_TILES = 512;                  // vocabulary <= 65536
constexpr size_t NA_SLOT_BYTES = (size_t)NA_GRID * 2 * SLOT_FLOATS * sizeof(float);
constexpr size_t NA_OFF_COUNTERS = NA_SLOT_BYTES;
constexpr size_t NA_OFF_STATUS = NA_OFF_COUNTERS + 2 * NA_MAX_TILES * sizeof(int);   // published + finished counters
constexpr size_t NA_OFF_TMAX = NA_OFF_STATUS + 256;
constexpr size_t NA_OFF_TARG = NA_OFF_TMAX + (size_t)NA_MAX_TILES * OURO_MAX_ROWS * sizeof(float);
constexpr size_t NA_BYTES = NA_OFF_TARG + (size_t)NA_MAX_TILES * OURO_MAX_ROWS * sizeof(int);
static_assert(NA_BYTES <= (5u << 20), "the static scratch is documented as 5 MiB");
constexpr int NA_MAX_DEVICES = 64;
}  // namespace

static __device__ __align__(256) unsigned char g_static_scratch[NA_BYTES];

namespace {
unsigned char *g_na_ptr[NA_MAX_DEVICES] = {};      // device address of g_static_scratch, per device
int g_na_smem[NA_MAX_DEVICES] = {};

// Once per device, with that device current: resolve the array's device address and size the kernel's
// shared memory.  Returns OURO_OK or an error with a text for ouro_last_error(NULL).
int na_setup(int dev) {
  if (g_na_ptr[dev]) return OURO_OK;
  void *ptr = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
  if (e != cudaSuccess || !ptr) {
    ouro_set_global_error(std::string("cudaGetSymbolAddress(static scratch): ") + cudaGetErrorString(e));
    return OURO_ECUDA;
  }
  int smem = 0;
  if ((e = cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess ||
      (e = cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) {
    ouro_set_global_error(std::string("static-scratch set-up: ") + cudaGetErrorString(e));
    return OURO_ECUDA;
  }
  if (!g_encode) {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn) {
      ouro_set_global_error("cuTensorMapEncodeTiled unavailable");
      return OURO_ECUDA;
    }
    g_encode = (EncodeTiledFn)fn;
  }
  g_na_smem[dev] = smem;
  g_na_ptr[dev] = (unsigned char *)ptr;
  return OURO_OK;
}
}  // namespace

extern "C" int ouro_lm_head_static(const void *x_dev, const void *lm_head_dev, int32_t rows, int32_t d_model, int32_t vocab,
                                   int32_t *argmax_dev, float *logits_dev, void *cuda_stream) {
  if (!x_dev || !lm_head_dev || !argmax_dev) {
    ouro_set_global_error("ouro_lm_head_static: null pointer");
    return OURO_EINVAL;
  }
  if (rows < 1 || rows > OURO_MAX_ROWS || d_model < 64 || d_model % 64 != 0 || vocab < 8 || vocab % 8 != 0 ||
      (vocab + TILE_N - 1) / TILE_N > NA_MAX_TILES || (((uintptr_t)x_dev | (uintptr_t)lm_head_dev) & 15)) {
    ouro_set_global_error("ouro_lm_head_static: size beyond the static scratch (rows 1..128, d_model a multiple of 64, "
                          "vocab a multiple of 8 and at most 65536) or pointers not 16-byte aligned");
    return OURO_EINVAL;
  }
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NA_MAX_DEVICES) {
    ouro_set_global_error("ouro_lm_head_static: no usable current device");
    return OURO_ECUDA;
  }
  int rc = na_setup(dev);
  if (rc != OURO_OK) return rc;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  unsigned char *base = g_na_ptr[dev];
  const int tiles = (vocab + TILE_N - 1) / TILE_N;
  // the array keeps whatever the last call left: counters and status must start at zero
  cudaError_t e = cudaMemsetAsync(base + NA_OFF_COUNTERS, 0, NA_OFF_TMAX - NA_OFF_COUNTERS, s);
  ChainParams cp{};
  cp.n = 1;
  GemmParams &p = cp.g[0];
  const int t_pad = (rows + 15) & ~15;
  if (e != cudaSuccess || !make_map(&p.a[0], lm_head_dev, vocab, d_model, TILE_N) || !make_map(&p.b, x_dev, rows, d_model, t_pad)) {
    ouro_set_global_error("ouro_lm_head_static: could not describe the operands to the copy engine");
    return OURO_ECUDA;
  }
  p.a_tiles[0] = tiles; p.a_rows[0] = vocab; p.a_count = 1;
  p.mode = MODE_HEAD;
  p.tiles = tiles;
  p.kb = d_model / BLOCK_K;
  p.t_pad = t_pad;
  p.rows = rows;
  p.stages = stages_for(t_pad, g_na_smem[dev]);
  p.out_f32 = logits_dev;
  p.ldo = vocab;
  p.tile_max = (float *)(base + NA_OFF_TMAX);
  p.tile_arg = (int *)(base + NA_OFF_TARG);
  p.wait_limit = 1u << 22;
  p.scratch = (float *)base;
  p.counters = (int *)(base + NA_OFF_COUNTERS);
  p.gen = 1;                                   // the words were cleared just above
  p.status = (int *)(base + NA_OFF_STATUS);
  const int total = tiles * p.kb;
  gemm_tc_kernel<<<total < NA_GRID ? total : NA_GRID, THREADS, g_na_smem[dev], s>>>(cp);
  argmax_tiles_kernel<<<rows, 128, 0, s>>>(p.tile_max, p.tile_arg, tiles, argmax_dev);
  int status = 0;
  if ((e = cudaGetLastError()) != cudaSuccess ||
      (e = cudaMemcpyAsync(&status, p.status, sizeof(int), cudaMemcpyDeviceToHost, s)) != cudaSuccess ||
      (e = cudaStreamSynchronize(s)) != cudaSuccess) {
    ouro_set_global_error(std::string("ouro_lm_head_static: ") + cudaGetErrorString(e));
    return OURO_ECUDA;
  }
  if (status != 0) {
    ouro_set_global_error("ouro_lm_head_static: a bounded device-side wait gave up");
    return OURO_ETIMEOUT;
  }
  return OURO_OK;
}
