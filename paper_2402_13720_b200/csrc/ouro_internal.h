// Internal declarations shared by the translation units of libouro (not part of the public ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <utility>
#include <vector>

#include "ouro.h"

typedef unsigned long long u64;

extern unsigned long long g_ouro_launches;   // kernels launched by this library since it was loaded
#define OURO_COUNT_LAUNCH() (++g_ouro_launches)

// Programmatic dependent launch: a kernel launched with launch_pdl may start while its predecessor in the
// stream is still draining.  Everything it does before pdl_wait() must be independent of earlier kernels
// (set-up, prefetch of weights); pdl_wait() returns once the predecessor has completed and its writes are
// visible.  pdl_trigger() lets the successor begin its own independent prologue.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
#endif

// Device-resident scalars of one decoding stream.
struct DevState {
  int32_t pending;   // last accepted token; its K/V is not cached yet (block row 0 of the next step)
  int32_t n_seq;     // tokens of the text recorded in seq_dev (== target cache length + 1)
  int32_t n_cand;    // candidates found by the last lookup (K' <= K)
  int32_t n_rows;    // rows of the last assembled target block
  int32_t A;         // accurate draft prefix of the last verification (Eq. 3)
  int32_t chosen;    // chosen candidate or -1
  int32_t m;         // matched suffix tokens of the chosen candidate (hat-A - 1, Eq. 9)
  int32_t n_acc;     // tokens accepted by the last verification
  int32_t accepted[OURO_MAX_GAMMA + OURO_MAX_BETA];
  int32_t status;    // sticky device-side error word (0 = fine)
  int32_t n_cand_last;  // copy of n_cand taken at acceptance (the acceptance record A .. n_cand_last is read back as one piece)
  u64 clock;         // phrase-pool stamp counter
  // last phrase-level drafting round of the draft model (Section 3.1)
  int32_t d_keep;    // draft tokens the round added (at most what was still missing of gamma)
  int32_t d_cached;  // how many of them have their K/V in the draft cache (matched suffix tokens kept)
  int32_t win_valid; // the lookahead window holds guesses (0 after a reset: the next draft forward fills it from the text)
};

// Per-row description of a query block.  Row r attends, in this order, cache slots [0, lin_end[r])
// and then slots [seg_start[r], seg_start[r] + seg_len[r]): the "virtual position" p of a key maps
// to slot p (p < lin_end) or seg_start + p - lin_end.  A trunk row has seg_len == 0; the suffix row
// (j, i) of Eq. 8 has lin_end = L + gamma + 1 and its own candidate's first i suffix slots.
struct BlockDev {
  int32_t *tok, *pos, *group, *lin_end, *seg_start, *seg_len;
  u64 *mask;  // [rows][2] visibility inside the block, for inspection only (kernels use the ranges)
};

struct PoolDev {
  int32_t *key;   // [sets*ways], -1 = free
  int32_t *suf;   // [sets*ways, S]
  u64 *stamp;     // [sets*ways]
  int32_t sets, ways, S;
};

struct ModelRt {
  bool present = false;
  ouro_model_desc d{};
  const void *embed = nullptr, *final_norm = nullptr, *lm_head = nullptr;
  std::vector<const void *> attn_norm, wq, wk, wv, wo, ffn_norm, w_gate, w_up, w_down;
  void *k_cache = nullptr, *v_cache = nullptr;
  float *rope_cos = nullptr, *rope_sin = nullptr;  // [max_seq, head_dim/2], filled at create
  BlockDev blk{};
  int32_t L = 0;        // cache length (host mirror)
  int32_t blk_rows = 0; // rows of the current block (0 = none assembled)
  int32_t blk_L = -1;   // cache length the block was assembled for
  bool blk_is_candidate = false;
  bool blk_rows_dev = false;  // blk_rows is an upper bound; the true count is DevState::n_rows (tensor-core path only)
};

struct Activations {  // sized for OURO_MAX_ROWS rows of the larger model
  float *x;        // residual stream [rows, d_model]
  void *xn;        // normed activations [rows, d_model], model dtype
  float *qkv;      // [rows, d_q + 2 d_kv]
  void *q;         // rotated queries [rows, d_q], model dtype
  void *att;       // attention output [rows, d_q], model dtype
  void *act;       // SwiGLU output [rows, d_ffn], model dtype
  float *logits;   // [rows, vocab]
  int32_t *argmax; // [rows]
  float *scratch;  // split-K partial sums / split-KV partial softmax states
  size_t scratch_bytes;
};

struct ouro_fast;   // tensor maps and launch state of the tensor-core paths (gemm_tc.cu)

struct ouro_ctx {
  ouro_fast *fast = nullptr;
  ModelRt m[2];
  ouro_params p{};
  cudaStream_t stream = nullptr;
  Activations a{};
  DevState *st = nullptr;
  int32_t *seq_dev = nullptr;     // [max_seq of target]
  int32_t *cand_suffix = nullptr; // [K, S]
  int32_t *cand_count = nullptr;  // [1]
  int32_t *draft_dev = nullptr;   // [gamma]
  int32_t *win_dev = nullptr;     // [OURO_MAX_WINDOW] lookahead window of the draft model
  PoolDev pool{};
  // host side
  std::vector<int32_t> seq;       // the text: prompt + accepted tokens (last one pending)
  int32_t *pin = nullptr;         // pinned host staging (PIN_INTS ints)
  // Mailbox in mapped pinned memory: the result the host needs in every step (the acceptance record) is written there
  // by the kernel itself, payload first, then a sequence number the host polls.
  int32_t *mbox = nullptr, *mbox_dev = nullptr;
  int32_t mseq = 0;
  const int *cur_rows_dev = nullptr;   // during a forward: where the kernels read the block's true row count, or NULL
  ouro_drafter_fn drafter = nullptr;
  void *drafter_user = nullptr;
  int32_t step = 0;
  std::string err;
  cudaEvent_t ev[6] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
  // per-kernel-class timing (ouro_profile_*)
  int prof_class = -1;
  std::vector<cudaEvent_t> prof_ev;
  size_t prof_used = 0;
  double prof_ms = 0.0;
  long prof_launches = 0;
};
void ouro_fast_teardown(ouro_ctx *c);
void prof_mark(ouro_ctx *c, int kernel_class);   // call before and after the launches of a class
struct ProfScope {
  ouro_ctx *c; int k;
  ProfScope(ouro_ctx *c_, int k_) : c(c_), k(k_) { if (c->prof_class == k) prof_mark(c, k); }
  ~ProfScope() { if (c->prof_class == k) prof_mark(c, k); }
};
enum { PIN_INTS = 1024 };

// ---- kernel launchers (kernels_block.cu) ---------------------------------------------------------
void launch_pool_clear(const PoolDev &P, DevState *st, cudaStream_t s);
void launch_pool_lookup(const PoolDev &P, const int32_t *key_dev, int key_index, int32_t key_value, int K,
                        int32_t *suffix, int32_t *count, cudaStream_t s);
void launch_pool_update(const PoolDev &P, DevState *st, const int32_t *ngrams, int n, int beta, int stride,
                        cudaStream_t s);
void launch_vanilla_accept(DevState *st, const int32_t *o, int32_t *seq_dev, cudaStream_t s);
void launch_assemble_candidates(const BlockDev &b, DevState *st, const int32_t *draft, const int32_t *suffix,
                                const int32_t *count, int L, int gamma, int S, int K, cudaStream_t s);
void launch_assemble_causal(const BlockDev &b, const int32_t *tokens, int n, int L, cudaStream_t s);
void launch_lookup_assemble(const PoolDev &P, const BlockDev &b, DevState *st, const int32_t *draft, int32_t *suffix,
                            int32_t *count, int L, int gamma, int S, int K, cudaStream_t s);
void launch_accept_compact_harvest(const BlockDev &b, DevState *st, const PoolDev &P, const int32_t *o, int32_t *seq_dev,
                                   const ouro_model_desc &d, void *k_cache, void *v_cache, int L, int gamma, int S,
                                   unsigned flags, int32_t *mbox, int32_t seq, cudaStream_t s);
enum { MBOX_INTS = 128, MBOX_ACCEPT = 16 };   // mailbox slot [flag, acceptance record]
void launch_draft_lookup_assemble(const PoolDev &P, const BlockDev &b, DevState *st, const int32_t *tokens, int n,
                                  int32_t *suffix, int32_t *count, int L, int S, int K, cudaStream_t s);
void launch_draft_accept_compact(const BlockDev &b, DevState *st, const int32_t *o, int32_t *out_dev, int have, int gamma,
                                 const ouro_model_desc &d, void *k_cache, void *v_cache, int L, int n, int S,
                                 cudaStream_t s);
void launch_draft_window_assemble(const BlockDev &b, DevState *st, const int32_t *tokens, int n, int32_t *win, int W,
                                  const int32_t *seq_dev, int L, cudaStream_t s);
void launch_draft_window_harvest(const BlockDev &b, DevState *st, const PoolDev &P, const int32_t *o, int32_t *out_or_null,
                                 int n, int W, int32_t *win, cudaStream_t s);
void launch_argmax(const float *logits, int rows, int vocab, int32_t *out, cudaStream_t s);
void launch_pick_token(const int32_t *src, int index, int32_t *dst, cudaStream_t s);
void launch_set_state(DevState *st, int32_t *seq_dev, int n_seq, int pending, int fill, cudaStream_t s);

// ---- kernel launchers (kernels_layer.cu) ---------------------------------------------------------
struct GemmSegs {  // up to three weight matrices [n_i, K] stacked along the output dimension
  const void *w[3];
  int n[3];
  int count;
};
enum { EPI_STORE = 0, EPI_RESIDUAL = 1 };
void launch_rope_table(float *cos_t, float *sin_t, int max_seq, int head_dim, float theta, cudaStream_t s);
void launch_embed(int dtype, const void *E, const int32_t *tok, int rows, int d, float *x, cudaStream_t s);
void launch_rmsnorm(int dtype, const float *x, const void *g, int rows, int d, float eps, void *out, cudaStream_t s);
void launch_gemm_simple(int dtype, const void *X, const GemmSegs &W, int rows, int K, float *Y, int ldy, int epi,
                        cudaStream_t s);
void launch_gemm_swiglu_simple(int dtype, const void *X, const void *Wg, const void *Wu, int rows, int K, int F,
                               void *act, cudaStream_t s);
void launch_rope_append(const ouro_model_desc &d, const float *qkv, const int32_t *pos, const float *cos_t,
                        const float *sin_t, int rows, int L, int layer, void *q, void *k_cache, void *v_cache,
                        cudaStream_t s);
void launch_attention_simple(const ouro_model_desc &d, const void *q, const void *k_cache, const void *v_cache,
                             const BlockDev &b, int rows, int layer, void *out, cudaStream_t s);

// ---- attn_tc.cu --------------------------------------------------------------------------------
bool attention_tc_supported(const ouro_model_desc &d);
size_t attention_tc_scratch_bytes(const ouro_model_desc &d);
int attention_tc_setup();
// Both return true when the spans still have to be folded by the kernel that consumes `out` (attn_fold.cuh).
bool launch_attention_tc(const ouro_model_desc &d, const void *q, const void *k_cache, const void *v_cache, const BlockDev &b,
                         int rows, int L, int n_vis_max, int layer, float *part, void *out, const int *rows_dev, cudaStream_t s);

// ---- attn_tm.cu (tcgen05 path, head dim 128) ---------------------------------------------------
bool attention_tm_supported(const ouro_model_desc &d);
int attention_tm_setup();
// Weights the kernels after the attention stream first (the output projection, the head of the gate and up matrices):
// the attention kernel leaves most of the HBM bandwidth unused, so its CTAs ask for these bytes to be brought into L2
// meanwhile.  Every region is a multiple of 16 bytes at a 16-byte aligned address; bytes 0 = no region.
struct L2Prefetch {
  const void *ptr[3] = {nullptr, nullptr, nullptr};
  size_t bytes[3] = {0, 0, 0};
};
bool launch_attention_tm(const ouro_model_desc &d, const void *q, const void *kmap, const void *vmap, const void *k_cache,
                         const void *v_cache, const BlockDev &b, int rows, int L, int n_vis_max, int layer, float *part,
                         void *out, int *status, const int *rows_dev, const L2Prefetch &pf, cudaStream_t s);
