// Integer side of one Ouroboros step: phrase pool, candidate packing, greedy acceptance,
// KV compaction, phrase harvest, row argmax.  All latency-bound kernels of one warp or one block.
#include "ouro_internal.h"

#define FULL 0xffffffffu

// ------------------------------------------------------------------------------- phrase pool
// sets x ways table; a phrase lives in the set selected by its first token (Section 3.2: phrases are
// retrieved by the draft's last token).  One warp works on one set, lanes stride over the ways.
// Every insert or refresh takes the next value of a global counter as stamp; stamps are unique.

__device__ __forceinline__ int pool_set(const PoolDev &P, int32_t key) {
  int bits = 31 - __clz(P.sets);
  return bits ? (int)(((uint32_t)key * 2654435761u) >> (32 - bits)) : 0;
}

__device__ __forceinline__ int warp_min_int(int v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v = min(v, __shfl_xor_sync(FULL, v, o));
  return v;
}

// way holding exactly this phrase, or INT_MAX.  phrase[] is warp-uniform.
__device__ int pool_find(const PoolDev &P, int set, const int32_t *phrase) {
  int lane = threadIdx.x & 31, best = INT_MAX;
  for (int w = lane; w < P.ways; w += 32) {
    int e = set * P.ways + w;
    bool hit = P.key[e] == phrase[0];
    for (int i = 0; hit && i < P.S; ++i) hit = P.suf[(size_t)e * P.S + i] == phrase[1 + i];
    if (hit) best = min(best, w);
  }
  return warp_min_int(best);
}

__device__ void pool_insert(const PoolDev &P, DevState *st, const int32_t *phrase) {
  int lane = threadIdx.x & 31;
  int set = pool_set(P, phrase[0]);
  int w = pool_find(P, set, phrase);
  if (w == INT_MAX) {
    int free_w = INT_MAX;
    u64 old = ~0ull;
    int old_w = INT_MAX;
    for (int c = lane; c < P.ways; c += 32) {
      int e = set * P.ways + c;
      if (P.key[e] < 0) {
        free_w = min(free_w, c);
      } else if (P.stamp[e] < old) {
        old = P.stamp[e];
        old_w = c;
      }
    }
    free_w = warp_min_int(free_w);
    if (free_w != INT_MAX) {
      w = free_w;
    } else {  // least recently stamped entry of the set
#pragma unroll
      for (int o = 16; o; o >>= 1) {
        u64 s2 = __shfl_xor_sync(FULL, old, o);
        int w2 = __shfl_xor_sync(FULL, old_w, o);
        if (s2 < old) { old = s2; old_w = w2; }
      }
      w = old_w;
    }
  }
  __syncwarp();
  if (lane == 0) {
    int e = set * P.ways + w;
    P.key[e] = phrase[0];
    for (int i = 0; i < P.S; ++i) P.suf[(size_t)e * P.S + i] = phrase[1 + i];
    P.stamp[e] = ++st->clock;
  }
  __syncwarp();
}

__device__ void pool_erase(const PoolDev &P, const int32_t *phrase) {
  int set = pool_set(P, phrase[0]);
  int w = pool_find(P, set, phrase);
  __syncwarp();
  if (w != INT_MAX && (threadIdx.x & 31) == 0) P.key[set * P.ways + w] = -1;
  __syncwarp();
}

// Up to K suffixes of phrases starting with key, newest first.  Returns the number found.
__device__ int pool_lookup(const PoolDev &P, int32_t key, int K, int32_t *suffix_out) {
  int lane = threadIdx.x & 31;
  int set = pool_set(P, key);
  if (P.ways <= 32) {
    // One way per lane: key and stamp are read once, the K newest are picked with shuffles alone, and all their
    // suffixes are fetched together: two round trips to memory whatever K is.  (Stamps start at 1 and are unique.)
    u64 mine = 0;
    if (lane < P.ways) {
      const int e = set * P.ways + lane;
      if (P.key[e] == key) mine = P.stamp[e];
    }
    int found = 0, sel = -1;                       // lane f remembers the way of the f-th newest phrase
    for (; found < K; ++found) {
      u64 best = mine;
      int best_w = mine ? lane : -1;
#pragma unroll
      for (int o = 16; o; o >>= 1) {
        u64 s2 = __shfl_xor_sync(FULL, best, o);
        int w2 = __shfl_xor_sync(FULL, best_w, o);
        if (s2 > best) { best = s2; best_w = w2; }
      }
      if (best_w < 0) break;
      if (lane == best_w) mine = 0;
      if (lane == found) sel = best_w;
    }
    for (int idx0 = 0; idx0 < found * P.S; idx0 += 32) {
      const int idx = idx0 + lane, f = min(idx / P.S, found - 1);
      const int w = __shfl_sync(FULL, sel, f);
      if (idx < found * P.S) suffix_out[idx] = P.suf[(size_t)(set * P.ways + w) * P.S + (idx - f * P.S)];
    }
    return found;
  }
  u64 bound = ~0ull;
  int found = 0;
  for (; found < K; ++found) {
    u64 best = 0;
    int best_w = -1;
    for (int c = lane; c < P.ways; c += 32) {
      int e = set * P.ways + c;
      if (P.key[e] == key && P.stamp[e] < bound && P.stamp[e] > best) {
        best = P.stamp[e];
        best_w = c;
      }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      u64 s2 = __shfl_xor_sync(FULL, best, o);
      int w2 = __shfl_xor_sync(FULL, best_w, o);
      if (s2 > best) { best = s2; best_w = w2; }
    }
    if (best_w < 0) break;
    bound = best;
    for (int i = lane; i < P.S; i += 32) suffix_out[found * P.S + i] = P.suf[(size_t)(set * P.ways + best_w) * P.S + i];
  }
  return found;
}

__global__ void pool_clear_kernel(PoolDev P, DevState *st) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < P.sets * P.ways) {
    P.key[i] = -1;
    P.stamp[i] = 0;
  }
  if (i == 0) st->clock = 0;
}

__global__ void pool_lookup_kernel(PoolDev P, const int32_t *key_dev, int key_index, int32_t key_value, int K,
                                   int32_t *suffix, int32_t *count) {
  int32_t key = key_dev ? key_dev[key_index] : key_value;
  int n = (key < 0 || P.S == 0) ? 0 : pool_lookup(P, key, K, suffix);
  if (threadIdx.x == 0) *count = n;
}

// n beta-grams, the g-th starting at ngrams + g*stride (stride 1 = sliding windows over a text).
__global__ void pool_update_kernel(PoolDev P, DevState *st, const int32_t *ngrams, int n, int beta, int stride) {
  int32_t ph[OURO_MAX_BETA];
  for (int g = 0; g < n; ++g) {
    for (int i = 0; i < beta; ++i) ph[i] = ngrams[(size_t)g * stride + i];
    pool_insert(P, st, ph);
  }
}

void launch_pool_clear(const PoolDev &P, DevState *st, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  int n = P.sets * P.ways;
  pool_clear_kernel<<<(n + 255) / 256, 256, 0, s>>>(P, st);
}
void launch_pool_lookup(const PoolDev &P, const int32_t *key_dev, int key_index, int32_t key_value, int K,
                        int32_t *suffix, int32_t *count, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  pool_lookup_kernel<<<1, 32, 0, s>>>(P, key_dev, key_index, key_value, K, suffix, count);
}
void launch_pool_update(const PoolDev &P, DevState *st, const int32_t *ngrams, int n, int beta, int stride,
                        cudaStream_t s) {
  if (n <= 0) return;
  OURO_COUNT_LAUNCH();
  pool_update_kernel<<<1, 32, 0, s>>>(P, st, ngrams, n, beta, stride);
}

// --------------------------------------------------------------------------- candidate packing
// Eq. 7: rows [pending, d_1..d_gamma, p^1_2..beta, .., p^K'_2..beta].  Trunk row b: position L+b, sees
// slots [0, L+b].  Suffix row (j, i): position L+gamma+i, sees slots [0, L+gamma] and its own
// candidate's rows (j, 1..i), which sit at slots L+1+gamma+j*S .. (Eq. 8).
__device__ __forceinline__ void assemble_candidates_body(const BlockDev &b, DevState *st, const int32_t *draft,
                                                         const int32_t *suffix, const int32_t *count, int L, int gamma,
                                                         int S, int K) {
  int nc = S > 0 ? min(*count, K) : 0;
  int B = 1 + gamma + nc * S;
  int r = threadIdx.x;
  if (r == 0) {
    st->n_cand = nc;
    st->n_rows = B;
  }
  if (r >= B) return;
  u64 m0 = 0, m1 = 0;
  if (r <= gamma) {
    b.tok[r] = r == 0 ? st->pending : draft[r - 1];
    b.pos[r] = L + r;
    b.group[r] = 0;
    b.lin_end[r] = L + r + 1;
    b.seg_start[r] = 0;
    b.seg_len[r] = 0;
    for (int c = 0; c <= r; ++c) (c < 64 ? m0 : m1) |= 1ull << (c & 63);
  } else {
    int j = (r - 1 - gamma) / S, i = (r - 1 - gamma) % S + 1;
    b.tok[r] = suffix[j * S + i - 1];
    b.pos[r] = L + gamma + i;
    b.group[r] = 1 + j;
    b.lin_end[r] = L + gamma + 1;
    b.seg_start[r] = L + 1 + gamma + j * S;
    b.seg_len[r] = i;
    for (int c = 0; c <= gamma; ++c) (c < 64 ? m0 : m1) |= 1ull << (c & 63);
    for (int c = 1 + gamma + j * S; c <= r; ++c) (c < 64 ? m0 : m1) |= 1ull << (c & 63);
  }
  b.mask[2 * r] = m0;
  b.mask[2 * r + 1] = m1;
}

__global__ void assemble_candidates_kernel(BlockDev b, DevState *st, const int32_t *draft, const int32_t *suffix,
                                           const int32_t *count, int L, int gamma, int S, int K) {
  assemble_candidates_body(b, st, draft, suffix, count, L, gamma, S, K);
}

// Writes a result the host is polling for: payload first, then (system-wide fence between) the sequence number.
__device__ __forceinline__ void mbox_post(int32_t *slot, const int32_t *payload, int n, int32_t seq) {
  for (int i = 0; i < n; ++i) slot[1 + i] = payload[i];
  __threadfence_system();
  *(volatile int32_t *)slot = seq;
}

// Lookup with key d_gamma (warp 0) and packing in one launch.
__global__ void lookup_assemble_kernel(PoolDev P, BlockDev b, DevState *st, const int32_t *draft, int32_t *suffix,
                                       int32_t *count, int L, int gamma, int S, int K) {
  pdl_wait();            // launched while the kernel before it drains; it never lets its own successor start early (the
                         // forward's kernels read the block description before their dependency wait)
  if (threadIdx.x < 32) {
    int32_t key = draft[gamma - 1];
    int n = (key < 0 || P.S == 0) ? 0 : pool_lookup(P, key, K, suffix);
    if (threadIdx.x == 0) *count = n;
  }
  __syncthreads();
  assemble_candidates_body(b, st, draft, suffix, count, L, gamma, S, K);
}

__global__ void assemble_causal_kernel(BlockDev b, const int32_t *tokens, int n, int L) {
  int r = threadIdx.x;
  if (r >= n) return;
  b.tok[r] = tokens[r];
  b.pos[r] = L + r;
  b.group[r] = 0;
  b.lin_end[r] = L + r + 1;
  b.seg_start[r] = 0;
  b.seg_len[r] = 0;
  u64 m0 = 0, m1 = 0;
  for (int c = 0; c <= r; ++c) (c < 64 ? m0 : m1) |= 1ull << (c & 63);
  b.mask[2 * r] = m0;
  b.mask[2 * r + 1] = m1;
}

void launch_assemble_candidates(const BlockDev &b, DevState *st, const int32_t *draft, const int32_t *suffix,
                                const int32_t *count, int L, int gamma, int S, int K, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  assemble_candidates_kernel<<<1, OURO_MAX_ROWS, 0, s>>>(b, st, draft, suffix, count, L, gamma, S, K);
}
void launch_lookup_assemble(const PoolDev &P, const BlockDev &b, DevState *st, const int32_t *draft, int32_t *suffix,
                            int32_t *count, int L, int gamma, int S, int K, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  launch_pdl(lookup_assemble_kernel, 1, OURO_MAX_ROWS, 0, s, P, b, st, draft, suffix, count, L, gamma, S, K);
}
void launch_assemble_causal(const BlockDev &b, const int32_t *tokens, int n, int L, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  assemble_causal_kernel<<<1, OURO_MAX_ROWS, 0, s>>>(b, tokens, n, L);
}

// ------------------------------------------------------------------------------- acceptance
// Eq. 3: A = longest a with d_1..a equal to the target's outputs at rows 0..a-1.  Eq. 9 (only when
// A == gamma): candidate j's chain is o[gamma], then the outputs at its own suffix rows; m_j counts
// its leading suffix tokens equal to that chain; the largest m_j wins, earliest j on ties.  The step
// accepts the matched tokens plus the chain's next output.  One thread: a few dozen comparisons.
__device__ void accept_body(const BlockDev &b, DevState *st, const int32_t *o, int32_t *seq_dev, int gamma, int S) {
  int nc = st->n_cand, A = 0, n = 0;
  while (A < gamma && b.tok[1 + A] == o[A]) ++A;
  for (int i = 0; i < A; ++i) st->accepted[n++] = b.tok[1 + i];
  int chosen = -1, m = 0;
  int32_t bonus = o[A];
  if (A == gamma && nc > 0) {
    int best_m = -1;
    for (int j = 0; j < nc; ++j) {
      int base = 1 + gamma + j * S, mj = 0;
      int32_t v = o[gamma];
      while (mj < S && b.tok[base + mj] == v) {
        v = o[base + mj];
        ++mj;
      }
      if (mj > best_m) {
        best_m = mj;
        chosen = j;
        bonus = v;
      }
    }
    m = best_m;
    for (int i = 0; i < m; ++i) st->accepted[n++] = b.tok[1 + gamma + chosen * S + i];
  }
  st->accepted[n++] = bonus;
  st->n_cand_last = nc;
  st->A = A;
  st->chosen = chosen;
  st->m = m;
  st->n_acc = n;
  st->pending = bonus;
  int base = st->n_seq;
  for (int i = 0; i < n; ++i) seq_dev[base + i] = st->accepted[i];
  st->n_seq = base + n;
}

// ------------------------------------------------------------------------------ KV compaction
// Slots L..L+A (pending token and accepted draft) already sit where they belong.  An accepted suffix of
// candidate j sits at slots L+1+gamma+j*S+[0,m) and moves to L+1+gamma+[0,m).  Source and destination
// ranges never overlap (j*S >= S >= m), so all rows move in parallel (accept_compact_harvest_kernel below).
// ---------------------------------------------------------------------------------- harvest
// Pool updates after a verification (Section 3.3), serialised in a fixed order by one warp:
//  1. when the draft was fully accepted: every tried phrase (d_gamma, p^j_2..beta), j ascending, is
//     replaced by (d_gamma, o[gamma], o at suffix rows (j,1..S-1)), the target's own continuation under
//     that candidate's context; an unchanged phrase is just refreshed;
//  2. when it was not: for every trunk row s in the discarded region (A+1 <= s <= gamma-1) whose
//     following draft tokens agree with the target outputs for at least max(1, beta-2) positions, the
//     beta-gram (t_s, o_s, .., o_{s+beta-2}) is inserted;
//  3. extension: every beta-window of the text that ends inside the newly accepted tokens.
__device__ void harvest_body(const BlockDev &b, DevState *st, const PoolDev &P, const int32_t *o, const int32_t *seq_dev,
                             int gamma, int S, unsigned flags) {
  const int beta = S + 1;
  int32_t ph[OURO_MAX_BETA], old[OURO_MAX_BETA];
  int A = st->A, nc = st->n_cand;
  if ((flags & OURO_HARVEST_CANDIDATES) && A == gamma && nc > 0) {
    for (int j = 0; j < nc; ++j) {
      int base = 1 + gamma + j * S;
      old[0] = ph[0] = b.tok[gamma];
      bool same = true;
      for (int i = 0; i < S; ++i) {
        old[1 + i] = b.tok[base + i];
        ph[1 + i] = i == 0 ? o[gamma] : o[base + i - 1];
        same = same && old[1 + i] == ph[1 + i];
      }
      if (!same) pool_erase(P, old);
      pool_insert(P, st, ph);
    }
  }
  if ((flags & OURO_HARVEST_MATCHED) && A < gamma) {
    int need = max(1, beta - 2);
    for (int s = A + 1; s < gamma; ++s) {
      int r = 0;
      while (s + r + 1 <= gamma && b.tok[s + r + 1] == o[s + r]) ++r;
      if (r >= need) {
        ph[0] = b.tok[s];
        for (int q = 0; q < beta - 1; ++q) ph[1 + q] = o[s + q];
        pool_insert(P, st, ph);
      }
    }
  }
  if (flags & OURO_HARVEST_ACCEPTED) {
    int n = st->n_seq;  // already includes the accepted tokens
    for (int e = n - st->n_acc; e < n; ++e) {
      if (e - beta + 1 < 0) continue;
      for (int i = 0; i < beta; ++i) ph[i] = seq_dev[e - beta + 1 + i];
      pool_insert(P, st, ph);
    }
  }
}

// Acceptance, compaction and harvest in one launch.  Block 0: one thread accepts (Eq. 3, Eq. 9), then its first
// warp harvests.  Blocks 1..: one (layer, K or V, suffix slot) each; every such block re-derives the chosen
// candidate and its matched length from the block tokens and the outputs (a few dozen comparisons) instead of
// waiting for block 0, then moves its cache row if the row belongs to the accepted suffix.
__global__ void accept_compact_harvest_kernel(BlockDev b, DevState *st, PoolDev P, const int32_t *o, int32_t *seq_dev,
                                              unsigned char *k_cache, unsigned char *v_cache, int L, int gamma, int S,
                                              int max_seq, int row_bytes, unsigned flags, int32_t *mbox, int32_t seq) {
  pdl_wait();            // its blocks are in place while the kernel that writes `o` finishes
  if (blockIdx.x == 0) {
    if (threadIdx.x == 0) {
      accept_body(b, st, o, seq_dev, gamma, S);
      if (mbox) mbox_post(mbox + MBOX_ACCEPT, &st->A, 4 + OURO_MAX_GAMMA + OURO_MAX_BETA + 2, seq);   // A .. n_cand_last
    }
    __syncthreads();
    if (threadIdx.x < 32 && (flags & (OURO_HARVEST_MATCHED | OURO_HARVEST_CANDIDATES | OURO_HARVEST_ACCEPTED)))
      harvest_body(b, st, P, o, seq_dev, gamma, S, flags);
    return;
  }
  __shared__ int s_chosen, s_m;
  if (threadIdx.x == 0) {
    int nc = st->n_cand, A = 0, chosen = -1, best = -1;
    while (A < gamma && b.tok[1 + A] == o[A]) ++A;
    if (A == gamma)
      for (int j = 0; j < nc; ++j) {
        int base = 1 + gamma + j * S, mj = 0;
        int32_t v = o[gamma];
        while (mj < S && b.tok[base + mj] == v) { v = o[base + mj]; ++mj; }
        if (mj > best) { best = mj; chosen = j; }
      }
    s_chosen = chosen;
    s_m = best < 0 ? 0 : best;
  }
  __syncthreads();
  const int idx = blockIdx.x - 1, t = idx % S, ly = idx / S;       // ly = 2 * layer + (0: K, 1: V)
  if (s_chosen <= 0 || t >= s_m) return;                           // candidate 0 already sits next to the trunk
  unsigned char *base = ((ly & 1) ? v_cache : k_cache) + (size_t)(ly >> 1) * max_seq * row_bytes;
  const uint4 *src = (const uint4 *)(base + (size_t)(L + 1 + gamma + s_chosen * S + t) * row_bytes);
  uint4 *dst = (uint4 *)(base + (size_t)(L + 1 + gamma + t) * row_bytes);
  for (int i = threadIdx.x; i < row_bytes / 16; i += blockDim.x) dst[i] = src[i];
}

void launch_accept_compact_harvest(const BlockDev &b, DevState *st, const PoolDev &P, const int32_t *o, int32_t *seq_dev,
                                   const ouro_model_desc &d, void *k_cache, void *v_cache, int L, int gamma, int S,
                                   unsigned flags, int32_t *mbox, int32_t seq, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  const int es = d.dtype == OURO_BF16 ? 2 : 4;
  launch_pdl(accept_compact_harvest_kernel, 1 + S * d.n_layers * 2, 128, 0, s, b, st, P, o, seq_dev, (unsigned char *)k_cache,
             (unsigned char *)v_cache, L, gamma, S, (int)d.max_seq, d.n_kv_heads * d.head_dim * es, flags, mbox, seq);
}

// ------------------------------------------------------------- phrase-level drafting (Section 3.1)
// A drafting round of the draft model.  Rows 0..n-1 are text it is fed (tokens[0..n-1], no verification needed),
// then the suffixes of up to K pool phrases that start with tokens[n-1], packed as in Eq. 7 / Eq. 8 with the
// n text rows in the role of the trunk.
__global__ void draft_lookup_assemble_kernel(PoolDev P, BlockDev b, DevState *st, const int32_t *tokens, int n,
                                             int32_t *suffix, int32_t *count, int L, int S, int K) {
  if (threadIdx.x < 32) {
    int32_t key = tokens[n - 1];
    int found = (key < 0 || P.S == 0 || S == 0) ? 0 : pool_lookup(P, key, K, suffix);
    if (threadIdx.x == 0) *count = found;
  }
  __syncthreads();
  const int nc = S > 0 ? min(*count, K) : 0, B = n + nc * S, r = threadIdx.x;
  if (r == 0) {
    st->n_cand = nc;
    st->n_rows = B;
  }
  if (r >= B) return;
  u64 m0 = 0, m1 = 0;
  if (r < n) {
    b.tok[r] = tokens[r];
    b.pos[r] = L + r;
    b.group[r] = 0;
    b.lin_end[r] = L + r + 1;
    b.seg_start[r] = 0;
    b.seg_len[r] = 0;
    for (int c = 0; c <= r; ++c) (c < 64 ? m0 : m1) |= 1ull << (c & 63);
  } else {
    const int j = (r - n) / S, i = (r - n) % S + 1;
    b.tok[r] = suffix[j * S + i - 1];
    b.pos[r] = L + n - 1 + i;
    b.group[r] = 1 + j;
    b.lin_end[r] = L + n;
    b.seg_start[r] = L + n + j * S;
    b.seg_len[r] = i;
    for (int c = 0; c < n; ++c) (c < 64 ? m0 : m1) |= 1ull << (c & 63);
    for (int c = n + j * S; c <= r; ++c) (c < 64 ? m0 : m1) |= 1ull << (c & 63);
  }
  b.mask[2 * r] = m0;
  b.mask[2 * r + 1] = m1;
}

// The round's outcome.  The draft model's next greedy token is o[n-1]; candidate j's chain continues from it as
// in Eq. 9; the longest match wins (earliest on ties) and the round yields its m tokens plus the chain's next
// one, cut to what the draft still lacks.  Block 0 writes the tokens; blocks 1.. each re-derive the choice and
// move one row of the draft cache next to the text (candidate 0 already sits there).
__global__ void draft_accept_compact_kernel(BlockDev b, DevState *st, const int32_t *o, int32_t *out_dev, int have,
                                            int gamma, unsigned char *k_cache, unsigned char *v_cache, int L, int n, int S,
                                            int max_seq, int row_bytes) {
  __shared__ int s_chosen, s_m;
  __shared__ int32_t s_bonus;
  if (threadIdx.x == 0) {
    const int nc = st->n_cand;
    int chosen = -1, best = -1;
    int32_t bonus = o[n - 1];
    for (int j = 0; j < nc; ++j) {
      int base = n + j * S, mj = 0;
      int32_t v = o[n - 1];
      while (mj < S && b.tok[base + mj] == v) { v = o[base + mj]; ++mj; }
      if (mj > best) { best = mj; chosen = j; bonus = v; }
    }
    s_chosen = chosen;
    s_m = best < 0 ? 0 : best;
    s_bonus = bonus;
  }
  __syncthreads();
  const int m = s_m, keep = min(m + 1, gamma - have), cached = min(m, keep);
  if (blockIdx.x == 0) {
    if (threadIdx.x < keep) out_dev[have + threadIdx.x] = (int)threadIdx.x < m ? b.tok[n + s_chosen * S + threadIdx.x] : s_bonus;
    if (threadIdx.x == 0) {
      st->d_keep = keep;
      st->d_cached = cached;
    }
    return;
  }
  const int idx = blockIdx.x - 1, t = idx % S, ly = idx / S;       // ly = 2 * layer + (0: K, 1: V)
  if (s_chosen <= 0 || t >= cached) return;
  unsigned char *base = ((ly & 1) ? v_cache : k_cache) + (size_t)(ly >> 1) * max_seq * row_bytes;
  const uint4 *src = (const uint4 *)(base + (size_t)(L + n + s_chosen * S + t) * row_bytes);
  uint4 *dst = (uint4 *)(base + (size_t)(L + n + t) * row_bytes);
  for (int i = threadIdx.x; i < row_bytes / 16; i += blockDim.x) dst[i] = src[i];
}

void launch_draft_lookup_assemble(const PoolDev &P, const BlockDev &b, DevState *st, const int32_t *tokens, int n,
                                  int32_t *suffix, int32_t *count, int L, int S, int K, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  draft_lookup_assemble_kernel<<<1, OURO_MAX_ROWS, 0, s>>>(P, b, st, tokens, n, suffix, count, L, S, K);
}
void launch_draft_accept_compact(const BlockDev &b, DevState *st, const int32_t *o, int32_t *out_dev, int have, int gamma,
                                 const ouro_model_desc &d, void *k_cache, void *v_cache, int L, int n, int S,
                                 cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  const int es = d.dtype == OURO_BF16 ? 2 : 4;
  draft_accept_compact_kernel<<<1 + (S > 0 ? S : 0) * d.n_layers * 2, 128, 0, s>>>(
      b, st, o, out_dev, have, gamma, (unsigned char *)k_cache, (unsigned char *)v_cache, L, n, S, d.max_seq,
      d.n_kv_heads * d.head_dim * es);
}

// ------------------------------------------- phrase generation during the draft forward (Section 3.1)
// A draft forward with a lookahead window: rows 0..n-1 are text the draft model is fed, rows n..n+W-1 hold the
// window's guesses for the W positions that follow, packed like one candidate suffix (window row i sees the text and
// window rows 1..i).  An empty window (after a reset) is first filled from the end of the text.
__global__ void draft_window_assemble_kernel(BlockDev b, DevState *st, const int32_t *tokens, int n, int32_t *win, int W,
                                             const int32_t *seq_dev, int L) {
  const int r = threadIdx.x;
  if (!st->win_valid) {
    const int n_seq = st->n_seq;
    if (r < W) {
      const int src = n_seq - W + r;                      // the text's last W tokens; a short text repeats its last one in front
      win[r] = seq_dev[src >= 0 ? src : n_seq - 1];
    }
  }
  __syncthreads();
  if (r == 0) {
    st->win_valid = 1;
    st->n_cand = W > 0 ? 1 : 0;
    st->n_rows = n + W;
  }
  if (r >= n + W) return;
  u64 m0 = 0, m1 = 0;
  if (r < n) {
    b.tok[r] = tokens[r];
    b.pos[r] = L + r;
    b.group[r] = 0;
    b.lin_end[r] = L + r + 1;
    b.seg_start[r] = 0;
    b.seg_len[r] = 0;
    for (int c = 0; c <= r; ++c) (c < 64 ? m0 : m1) |= 1ull << (c & 63);
  } else {
    const int i = r - n + 1;
    b.tok[r] = win[i - 1];
    b.pos[r] = L + n - 1 + i;
    b.group[r] = 1;
    b.lin_end[r] = L + n;
    b.seg_start[r] = L + n;
    b.seg_len[r] = i;
    for (int c = 0; c <= r; ++c) (c < 64 ? m0 : m1) |= 1ull << (c & 63);
  }
  b.mask[2 * r] = m0;
  b.mask[2 * r + 1] = m1;
}

// After that forward: chain[0] = o[n-1] is the next draft token; chain[i] = o[n-1+i] is the prediction after window
// guess i.  The beta-grams along the diagonal, (src[i], chain[i], .., chain[i+S-1]) for i = 0 .. W-S+1 with src[0] the
// last text token and src[i] guess i, enter the pool in that order; then the window becomes chain[1..W].
__global__ void draft_window_harvest_kernel(BlockDev b, DevState *st, PoolDev P, const int32_t *o, int32_t *out, int n, int W,
                                            int32_t *win) {
  const int lane = threadIdx.x, S = P.S;
  int32_t ph[OURO_MAX_BETA];
  if (S >= 1)
    for (int i = 0; i + S - 1 <= W; ++i) {
      ph[0] = b.tok[n - 1 + i];
      for (int q = 0; q < S; ++q) ph[1 + q] = o[n - 1 + i + q];
      pool_insert(P, st, ph);
    }
  __syncwarp();
  const int32_t next = lane < W ? o[n + lane] : 0;
  __syncwarp();
  if (lane < W) win[lane] = next;
  if (lane == 0 && out) *out = o[n - 1];
}

void launch_draft_window_assemble(const BlockDev &b, DevState *st, const int32_t *tokens, int n, int32_t *win, int W,
                                  const int32_t *seq_dev, int L, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  draft_window_assemble_kernel<<<1, OURO_MAX_ROWS, 0, s>>>(b, st, tokens, n, win, W, seq_dev, L);
}
void launch_draft_window_harvest(const BlockDev &b, DevState *st, const PoolDev &P, const int32_t *o, int32_t *out_or_null,
                                 int n, int W, int32_t *win, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  draft_window_harvest_kernel<<<1, 32, 0, s>>>(b, st, P, o, out_or_null, n, W, win);
}

// ----------------------------------------------------------------------------------- argmax
// Greedy choice per row; equal maxima resolve to the smallest token id.
__global__ void argmax_kernel(const float *logits, int vocab, int32_t *out) {
  const float *row = logits + (size_t)blockIdx.x * vocab;
  float best = -INFINITY;
  int idx = INT_MAX;
  for (int i = threadIdx.x; i < vocab; i += blockDim.x) {
    float v = row[i];
    if (v > best || (v == best && i < idx)) { best = v; idx = i; }
  }
  __shared__ float sv[32];
  __shared__ int si[32];
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    float v2 = __shfl_xor_sync(FULL, best, o);
    int i2 = __shfl_xor_sync(FULL, idx, o);
    if (v2 > best || (v2 == best && i2 < idx)) { best = v2; idx = i2; }
  }
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { sv[warp] = best; si[warp] = idx; }
  __syncthreads();
  if (warp == 0) {
    int nw = blockDim.x >> 5;
    best = lane < nw ? sv[lane] : -INFINITY;
    idx = lane < nw ? si[lane] : INT_MAX;
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      float v2 = __shfl_xor_sync(FULL, best, o);
      int i2 = __shfl_xor_sync(FULL, idx, o);
      if (v2 > best || (v2 == best && i2 < idx)) { best = v2; idx = i2; }
    }
    if (lane == 0) out[blockIdx.x] = idx == INT_MAX ? 0 : idx;
  }
}

void launch_argmax(const float *logits, int rows, int vocab, int32_t *out, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  argmax_kernel<<<rows, 256, 0, s>>>(logits, vocab, out);
}

// Plain greedy decoding: the row-0 output becomes the next pending token and joins the text.
__global__ void vanilla_accept_kernel(DevState *st, const int32_t *o, int32_t *seq_dev) {
  st->pending = o[0];
  seq_dev[st->n_seq] = o[0];
  st->n_seq += 1;
}
void launch_vanilla_accept(DevState *st, const int32_t *o, int32_t *seq_dev, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  vanilla_accept_kernel<<<1, 1, 0, s>>>(st, o, seq_dev);
}

__global__ void pick_token_kernel(const int32_t *src, int index, int32_t *dst) { *dst = src[index]; }
void launch_pick_token(const int32_t *src, int index, int32_t *dst, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  pick_token_kernel<<<1, 1, 0, s>>>(src, index, dst);
}

// Text of n_seq tokens ending in the pending token; with fill, the earlier positions are recorded as 0.
__global__ void set_state_kernel(DevState *st, int32_t *seq_dev, int n_seq, int pending, int fill) {
  if (fill)
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_seq - 1; i += gridDim.x * blockDim.x) seq_dev[i] = 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    seq_dev[n_seq - 1] = pending;
    st->pending = pending;
    st->n_seq = n_seq;
    st->n_cand = 0;
    st->n_rows = 0;
    st->status = 0;
    st->win_valid = 0;
  }
}
void launch_set_state(DevState *st, int32_t *seq_dev, int n_seq, int pending, int fill, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  set_state_kernel<<<8, 256, 0, s>>>(st, seq_dev, n_seq, pending, fill);
}
