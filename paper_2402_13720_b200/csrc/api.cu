// C ABI of libouro: context set-up, the model forward as a chain of kernel launches, and the host
// loops of Ouroboros and of plain greedy decoding.  See include/ouro.h for the contract of each call.
#include <algorithm>
#include <atomic>
#include <chrono>
#include <cstdio>
#include <cstring>
#include <new>

#include "ouro_internal.h"

static thread_local std::string g_create_err;
unsigned long long g_ouro_launches = 0;
extern "C" uint64_t ouro_kernel_launches(void) { return g_ouro_launches; }

static int fail(ouro_ctx *c, int code, const std::string &msg) {
  if (c) c->err = msg; else g_create_err = msg;
  return code;
}
#define CK(call)                                                                                     \
  do {                                                                                               \
    cudaError_t e_ = (call);                                                                         \
    if (e_ != cudaSuccess)                                                                           \
      return fail(c, OURO_ECUDA, std::string(#call) + ": " + cudaGetErrorString(e_));               \
  } while (0)
#define CKL() CK(cudaGetLastError())
#define TRY(expr)                                                                                    \
  do {                                                                                               \
    int rc_ = (expr);                                                                                \
    if (rc_ != OURO_OK) return rc_;                                                                  \
  } while (0)

extern "C" const char *ouro_strerror(int s) {
  switch (s) {
    case OURO_OK: return "ok";
    case OURO_EINVAL: return "invalid argument";
    case OURO_ENOMEM: return "workspace too small or host allocation failed";
    case OURO_ECAPACITY: return "KV cache or block row capacity exceeded";
    case OURO_ECUDA: return "CUDA call failed";
    case OURO_ETIMEOUT: return "a bounded device-side wait gave up";
    case OURO_ESTATE: return "call order violated";
  }
  return "unknown status";
}
void ouro_set_global_error(const std::string &msg) { g_create_err = msg; }   // text for calls that have no context
extern "C" const char *ouro_last_error(const ouro_ctx *c) { return c ? c->err.c_str() : g_create_err.c_str(); }

// ---------------------------------------------------------------------------- workspace layout
struct Carver {
  char *base;
  size_t off;
  template <typename T> T *take(size_t n) {
    off = (off + 255) & ~(size_t)255;
    T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
    off += n * sizeof(T);
    return p;
  }
};

static bool desc_ok(const ouro_model_desc *d) {
  return d && d->n_layers > 0 && d->d_model > 0 && d->d_model % 8 == 0 && d->n_heads > 0 && d->n_kv_heads > 0 &&
         d->n_heads % d->n_kv_heads == 0 && d->head_dim % 32 == 0 && d->head_dim >= 32 && d->head_dim <= 128 &&
         d->d_ffn > 0 && d->d_ffn % 8 == 0 && d->vocab > 0 && d->max_seq > 0 &&
         (d->dtype == OURO_F32 || d->dtype == OURO_BF16) && d->rope_theta > 0.f;
}
static bool params_ok(const ouro_params *p) {
  if (!p) return false;
  if (p->gamma < 1 || p->gamma > OURO_MAX_GAMMA || p->beta < 1 || p->beta > OURO_MAX_BETA) return false;
  if (p->K < 0 || p->K > OURO_MAX_K) return false;
  if (p->pool_sets < 1 || (p->pool_sets & (p->pool_sets - 1)) || p->pool_ways < 1) return false;
  if (p->window < 0 || p->window > OURO_MAX_WINDOW || (p->window > 0 && (p->flags & OURO_DRAFT_PHRASES))) return false;
  return 1 + p->gamma + p->K * (p->beta - 1) <= OURO_MAX_ROWS;
}

size_t ouro_scratch_bytes(const ouro_model_desc *t, const ouro_model_desc *d);  // gemm/attention scratch (fast paths)

// Lays out every device buffer of a context inside the workspace (or just measures when base is null).
static size_t carve(ouro_ctx *c, char *base, const ouro_model_desc *t, const ouro_model_desc *d, const ouro_params *p) {
  Carver cv{base, 0};
  const size_t R = OURO_MAX_ROWS;
  auto mx = [&](auto f) { return std::max<size_t>(f(t), d ? f(d) : 0); };
  size_t dm = mx([](const ouro_model_desc *m) { return (size_t)m->d_model; });
  size_t dq = mx([](const ouro_model_desc *m) { return (size_t)m->n_heads * m->head_dim; });
  size_t dqkv = mx([](const ouro_model_desc *m) { return (size_t)(m->n_heads + 2 * m->n_kv_heads) * m->head_dim; });
  size_t F = mx([](const ouro_model_desc *m) { return (size_t)m->d_ffn; });
  size_t V = mx([](const ouro_model_desc *m) { return (size_t)m->vocab; });
  Activations a{};
  a.x = cv.take<float>(R * dm);
  a.xn = cv.take<float>(R * dm);
  a.qkv = cv.take<float>(R * dqkv);
  a.q = cv.take<float>(R * dq);
  a.att = cv.take<float>(R * dq);
  a.act = cv.take<float>(R * F);
  a.logits = cv.take<float>(R * V);
  a.argmax = cv.take<int32_t>(R);
  a.scratch_bytes = ouro_scratch_bytes(t, d);
  a.scratch = cv.take<float>(a.scratch_bytes / 4);
  DevState *st = cv.take<DevState>(1);
  int32_t *seq_dev = cv.take<int32_t>((size_t)t->max_seq + OURO_MAX_ROWS);
  int S = p->beta - 1;
  int32_t *cand_suffix = cv.take<int32_t>((size_t)std::max(1, p->K * S));
  int32_t *cand_count = cv.take<int32_t>(1);
  int32_t *draft_dev = cv.take<int32_t>(p->gamma);
  int32_t *win_dev = cv.take<int32_t>(OURO_MAX_WINDOW);
  PoolDev pool{};
  size_t cap = (size_t)p->pool_sets * p->pool_ways;
  pool.key = cv.take<int32_t>(cap);
  pool.suf = cv.take<int32_t>(cap * std::max(1, S));
  pool.stamp = cv.take<u64>(cap);
  pool.sets = p->pool_sets;
  pool.ways = p->pool_ways;
  pool.S = S;
  const ouro_model_desc *ds[2] = {t, d};
  BlockDev blk[2]{};
  float *rc[2]{}, *rs[2]{};
  for (int w = 0; w < 2; ++w) {
    if (!ds[w]) continue;
    blk[w].tok = cv.take<int32_t>(R);
    blk[w].pos = cv.take<int32_t>(R);
    blk[w].group = cv.take<int32_t>(R);
    blk[w].lin_end = cv.take<int32_t>(R);
    blk[w].seg_start = cv.take<int32_t>(R);
    blk[w].seg_len = cv.take<int32_t>(R);
    blk[w].mask = cv.take<u64>(2 * R);
    size_t nt = (size_t)ds[w]->max_seq * (ds[w]->head_dim / 2);
    rc[w] = cv.take<float>(nt);
    rs[w] = cv.take<float>(nt);
  }
  if (c) {
    c->a = a;
    c->st = st;
    c->seq_dev = seq_dev;
    c->cand_suffix = cand_suffix;
    c->cand_count = cand_count;
    c->draft_dev = draft_dev;
    c->win_dev = win_dev;
    c->pool = pool;
    for (int w = 0; w < 2; ++w) {
      c->m[w].blk = blk[w];
      c->m[w].rope_cos = rc[w];
      c->m[w].rope_sin = rs[w];
    }
  }
  return (cv.off + 255) & ~(size_t)255;
}

extern "C" size_t ouro_workspace_bytes(const ouro_model_desc *t, const ouro_model_desc *d, const ouro_params *p) {
  if (!desc_ok(t) || (d && !desc_ok(d)) || !params_ok(p)) return 0;
  return carve(nullptr, nullptr, t, d, p);
}

static void bind_model(ModelRt &M, const ouro_model_desc *d, const ouro_model_mem *mem) {
  M.present = true;
  M.d = *d;
  M.embed = mem->embed;
  M.final_norm = mem->final_norm;
  M.lm_head = mem->lm_head;
  M.k_cache = mem->k_cache;
  M.v_cache = mem->v_cache;
  auto cp = [&](std::vector<const void *> &dst, const void *const *src) { dst.assign(src, src + d->n_layers); };
  cp(M.attn_norm, mem->attn_norm);
  cp(M.wq, mem->wq);
  cp(M.wk, mem->wk);
  cp(M.wv, mem->wv);
  cp(M.wo, mem->wo);
  cp(M.ffn_norm, mem->ffn_norm);
  cp(M.w_gate, mem->w_gate);
  cp(M.w_up, mem->w_up);
  cp(M.w_down, mem->w_down);
}

static bool mem_ok(const ouro_model_mem *m) {
  return m && m->embed && m->final_norm && m->lm_head && m->attn_norm && m->wq && m->wk && m->wv && m->wo &&
         m->ffn_norm && m->w_gate && m->w_up && m->w_down && m->k_cache && m->v_cache;
}

int ouro_fast_setup(ouro_ctx *c);  // tensor maps etc. of the tensor-core paths (gemm_tc.cu)
void ouro_fast_reset(ouro_ctx *c, bool force);   // clears split-K / chain counters (always, or only after a device-side give-up)
void ouro_fast_mark_dirty(ouro_ctx *c);
bool ouro_fast_available(ouro_ctx *c, int which);   // model `which` runs on the tensor-core kernels

extern "C" int ouro_create(const ouro_model_desc *t, const ouro_model_mem *tm, const ouro_model_desc *d,
                           const ouro_model_mem *dm, const ouro_params *p, void *ws, size_t ws_bytes, void *stream,
                           ouro_ctx **out) {
  ouro_ctx *c = nullptr;
  if (!out) return fail(c, OURO_EINVAL, "out is NULL");
  if (!desc_ok(t) || !mem_ok(tm)) return fail(c, OURO_EINVAL, "target description or memory invalid");
  if ((d != nullptr) != (dm != nullptr)) return fail(c, OURO_EINVAL, "draft description and memory must come together");
  if (d && (!desc_ok(d) || !mem_ok(dm))) return fail(c, OURO_EINVAL, "draft description or memory invalid");
  if (d && d->vocab != t->vocab) return fail(c, OURO_EINVAL, "draft and target vocabularies differ");
  if (!params_ok(p)) return fail(c, OURO_EINVAL, "decoding parameters invalid (gamma, beta, K, pool shape or rows > OURO_MAX_ROWS)");
  if (!ws || ((uintptr_t)ws & 255)) return fail(c, OURO_EINVAL, "workspace must be 256-byte aligned device memory");
  size_t need = carve(nullptr, nullptr, t, d, p);
  if (ws_bytes < need) return fail(c, OURO_ENOMEM, "workspace smaller than ouro_workspace_bytes()");
  ouro_ctx *n = new (std::nothrow) ouro_ctx();
  if (!n) return fail(c, OURO_ENOMEM, "host allocation failed");
  n->p = *p;
  n->stream = (cudaStream_t)stream;
  bind_model(n->m[OURO_TARGET], t, tm);
  if (d) bind_model(n->m[OURO_DRAFT], d, dm);
  carve(n, (char *)ws, t, d, p);
  auto bail = [&](int code, const std::string &msg) {
    g_create_err = msg;
    if (n->pin) cudaFreeHost(n->pin);
    if (n->mbox) cudaFreeHost(n->mbox);
    for (auto &e : n->ev) if (e) cudaEventDestroy(e);
    ouro_fast_teardown(n);
    delete n;
    return code;
  };
  cudaError_t e = cudaMallocHost((void **)&n->pin, PIN_INTS * sizeof(int32_t));
  if (e != cudaSuccess) return bail(OURO_ENOMEM, std::string("cudaMallocHost: ") + cudaGetErrorString(e));
  // the mailbox is optional: without mapped host memory the results come back by copy
  if (cudaHostAlloc((void **)&n->mbox, MBOX_INTS * sizeof(int32_t), cudaHostAllocMapped) == cudaSuccess) {
    memset(n->mbox, 0, MBOX_INTS * sizeof(int32_t));
    if (cudaHostGetDevicePointer((void **)&n->mbox_dev, n->mbox, 0) != cudaSuccess) {
      cudaFreeHost(n->mbox);
      n->mbox = n->mbox_dev = nullptr;
    }
  } else {
    n->mbox = nullptr;
    (void)cudaGetLastError();
  }
  for (auto &ev : n->ev)
    if ((e = cudaEventCreate(&ev)) != cudaSuccess) return bail(OURO_ECUDA, std::string("cudaEventCreate: ") + cudaGetErrorString(e));
  for (int w = 0; w < 2; ++w)
    if (n->m[w].present)
      launch_rope_table(n->m[w].rope_cos, n->m[w].rope_sin, n->m[w].d.max_seq, n->m[w].d.head_dim, n->m[w].d.rope_theta,
                        n->stream);
  // The attention kernels multiply masked keys' V rows by an exact zero, so rows nobody has written yet must not
  // hold NaN or infinity: the caches start out cleared.
  for (int w = 0; w < 2; ++w)
    if (n->m[w].present) {
      const ouro_model_desc &md = n->m[w].d;
      const size_t bytes = (size_t)md.n_layers * md.max_seq * md.n_kv_heads * md.head_dim * (md.dtype == OURO_BF16 ? 2 : 4);
      if ((e = cudaMemsetAsync(n->m[w].k_cache, 0, bytes, n->stream)) != cudaSuccess ||
          (e = cudaMemsetAsync(n->m[w].v_cache, 0, bytes, n->stream)) != cudaSuccess)
        return bail(OURO_ECUDA, std::string("clearing the KV cache: ") + cudaGetErrorString(e));
    }
  launch_pool_clear(n->pool, n->st, n->stream);
  launch_set_state(n->st, n->seq_dev, 1, 0, 1, n->stream);
  int rc = ouro_fast_setup(n);
  if (rc != OURO_OK) return bail(rc, n->err);
  if ((e = cudaStreamSynchronize(n->stream)) != cudaSuccess || (e = cudaGetLastError()) != cudaSuccess)
    return bail(OURO_ECUDA, std::string("set-up kernels: ") + cudaGetErrorString(e));
  n->seq.assign(1, 0);
  *out = n;
  return OURO_OK;
}

extern "C" int ouro_destroy(ouro_ctx *c) {
  if (!c) return OURO_EINVAL;
  cudaStreamSynchronize(c->stream);
  if (c->pin) cudaFreeHost(c->pin);
  if (c->mbox) cudaFreeHost(c->mbox);
  for (auto &e : c->ev) if (e) cudaEventDestroy(e);
  for (auto &e : c->prof_ev) cudaEventDestroy(e);
  ouro_fast_teardown(c);
  delete c;
  return OURO_OK;
}

static void forget_blocks(ouro_ctx *c) {
  for (auto &M : c->m) {
    M.blk_rows = 0;
    M.blk_L = -1;
  }
}

extern "C" int ouro_reset(ouro_ctx *c, int keep_pool) {
  if (!c) return OURO_EINVAL;
  c->m[0].L = c->m[1].L = 0;
  forget_blocks(c);
  c->seq.assign(1, 0);
  c->step = 0;
  ouro_fast_reset(c, true);
  launch_set_state(c->st, c->seq_dev, 1, 0, 1, c->stream);
  if (!keep_pool) launch_pool_clear(c->pool, c->st, c->stream);
  CKL();
  return OURO_OK;
}

extern "C" int ouro_set_state(ouro_ctx *c, int32_t cache_len, int32_t pending) {
  if (!c) return OURO_EINVAL;
  if (cache_len < 0 || cache_len + 1 > c->m[0].d.max_seq || (c->m[1].present && cache_len + 1 > c->m[1].d.max_seq))
    return fail(c, OURO_ECAPACITY, "cache_len does not fit max_seq");
  if (pending < 0 || pending >= c->m[0].d.vocab) return fail(c, OURO_EINVAL, "pending token out of range");
  c->m[0].L = c->m[1].L = cache_len;
  forget_blocks(c);
  c->seq.assign((size_t)cache_len + 1, 0);
  c->seq.back() = pending;
  c->step = 0;
  ouro_fast_reset(c, false);
  launch_set_state(c->st, c->seq_dev, cache_len + 1, pending, 1, c->stream);
  CKL();
  return OURO_OK;
}

extern "C" int ouro_get_state(ouro_ctx *c, int32_t *tl, int32_t *dl, int32_t *pending) {
  if (!c) return OURO_EINVAL;
  if (tl) *tl = c->m[0].L;
  if (dl) *dl = c->m[1].L;
  if (pending) *pending = c->seq.back();
  return OURO_OK;
}

extern "C" int ouro_set_drafter(ouro_ctx *c, ouro_drafter_fn fn, void *user) {
  if (!c) return OURO_EINVAL;
  c->drafter = fn;
  c->drafter_user = user;
  return OURO_OK;
}

// ------------------------------------------------------------------------------------ blocks
extern "C" int ouro_assemble_causal(ouro_ctx *c, int which, const int32_t *tokens_dev, int32_t n) {
  if (!c || which < 0 || which > 1 || !tokens_dev) return OURO_EINVAL;
  ModelRt &M = c->m[which];
  if (!M.present) return fail(c, OURO_ESTATE, "model not present");
  if (n < 1 || n > OURO_MAX_ROWS) return fail(c, OURO_ECAPACITY, "block rows outside 1..OURO_MAX_ROWS");
  if (M.L + n > M.d.max_seq) return fail(c, OURO_ECAPACITY, "cache length + block rows exceeds max_seq");
  launch_assemble_causal(M.blk, tokens_dev, n, M.L, c->stream);
  CKL();
  M.blk_rows = n;
  M.blk_rows_dev = false;
  M.blk_L = M.L;
  M.blk_is_candidate = false;
  return OURO_OK;
}

// Waits for a kernel to post sequence number `seq` in a mailbox slot.  The wait is bounded: after two seconds
// the stream is synchronised instead, which also surfaces a launch or execution error.
static int mbox_wait(ouro_ctx *c, int slot, int32_t seq) {
  volatile int32_t *flag = c->mbox + slot;
  const auto t0 = std::chrono::steady_clock::now();
  for (uint32_t spin = 0; *flag != seq; ++spin) {
    if ((spin & 4095) == 4095 && std::chrono::steady_clock::now() - t0 > std::chrono::seconds(2)) {
      CK(cudaStreamSynchronize(c->stream));
      if (*flag != seq) return fail(c, OURO_ECUDA, "a kernel finished without posting its result");
      break;
    }
  }
  std::atomic_thread_fence(std::memory_order_acquire);
  return OURO_OK;
}

extern "C" int ouro_assemble_candidates(ouro_ctx *c, const int32_t *draft_dev, const int32_t *suffix_dev,
                                        const int32_t *count_dev) {
  if (!c || !draft_dev || ((suffix_dev == nullptr) != (count_dev == nullptr))) return OURO_EINVAL;
  ModelRt &M = c->m[OURO_TARGET];
  const int gamma = c->p.gamma, S = c->p.beta - 1, K = c->p.K;
  if (M.L + 1 + gamma + K * S > M.d.max_seq) return fail(c, OURO_ECAPACITY, "cache length + block rows exceeds max_seq");
  if (!suffix_dev)
    launch_lookup_assemble(c->pool, M.blk, c->st, draft_dev, c->cand_suffix, c->cand_count, M.L, gamma, S, K, c->stream);
  else
    launch_assemble_candidates(M.blk, c->st, draft_dev, suffix_dev, count_dev, M.L, gamma, S, K, c->stream);
  CKL();
  if (ouro_fast_available(c, OURO_TARGET)) {
    // The tensor-core kernels read the block's row count from device memory: the forward is launched for the largest
    // block these parameters allow and the host never waits for the lookup.
    M.blk_rows = 1 + gamma + K * S;
    M.blk_rows_dev = true;
  } else {
    CK(cudaMemcpyAsync(c->pin, &c->st->n_rows, sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    M.blk_rows = c->pin[0];
    M.blk_rows_dev = false;
  }
  M.blk_L = M.L;
  M.blk_is_candidate = true;
  return OURO_OK;
}

extern "C" int ouro_block_get(ouro_ctx *c, int which, int32_t *tok, int32_t *pos, int32_t *group, uint64_t *mask,
                              int32_t *B) {
  if (!c || which < 0 || which > 1) return OURO_EINVAL;
  ModelRt &M = c->m[which];
  if (!M.present || M.blk_rows == 0) return fail(c, OURO_ESTATE, "no block assembled");
  CK(cudaStreamSynchronize(c->stream));
  if (M.blk_rows_dev) {                      // the host only knows an upper bound so far
    int32_t exact = 0;
    CK(cudaMemcpy(&exact, &c->st->n_rows, sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (exact < 1 || exact > M.blk_rows) return fail(c, OURO_ECUDA, "block has an impossible row count");
    M.blk_rows = exact;
    M.blk_rows_dev = false;
  }
  size_t n = M.blk_rows;
  if (tok) CK(cudaMemcpy(tok, M.blk.tok, n * 4, cudaMemcpyDeviceToHost));
  if (pos) CK(cudaMemcpy(pos, M.blk.pos, n * 4, cudaMemcpyDeviceToHost));
  if (group) CK(cudaMemcpy(group, M.blk.group, n * 4, cudaMemcpyDeviceToHost));
  if (mask) CK(cudaMemcpy(mask, M.blk.mask, n * 16, cudaMemcpyDeviceToHost));
  if (B) *B = M.blk_rows;
  return OURO_OK;
}

// --------------------------------------------------------------------------------- profiling
static void prof_flush(ouro_ctx *c) {
  if (c->prof_used == 0) return;
  cudaEventSynchronize(c->prof_ev[c->prof_used - 1]);
  for (size_t i = 0; i + 1 < c->prof_used; i += 2) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->prof_ev[i], c->prof_ev[i + 1]) == cudaSuccess) c->prof_ms += ms;
    c->prof_launches += 1;
  }
  c->prof_used = 0;
}
void prof_mark(ouro_ctx *c, int) {
  if (c->prof_used == c->prof_ev.size()) {
    if (c->prof_ev.size() >= 512) {
      prof_flush(c);
    } else {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return;
      c->prof_ev.push_back(e);
    }
  }
  cudaEventRecord(c->prof_ev[c->prof_used++], c->stream);
}
extern "C" int ouro_profile_enable(ouro_ctx *c, int kernel_class) {
  if (!c || kernel_class < OURO_PROF_OFF || kernel_class > OURO_PROF_GEMM) return OURO_EINVAL;
  prof_flush(c);
  c->prof_class = kernel_class;
  c->prof_ms = 0.0;
  c->prof_launches = 0;
  return OURO_OK;
}
extern "C" int ouro_profile_read(ouro_ctx *c, float *ms_total, int32_t *launches) {
  if (!c) return OURO_EINVAL;
  prof_flush(c);
  if (ms_total) *ms_total = (float)c->prof_ms;
  if (launches) *launches = (int32_t)c->prof_launches;
  return OURO_OK;
}

// ----------------------------------------------------------------------------------- forward
int ouro_fast_embed(ouro_ctx *c, int which, int rows);                     // embedding + first norm's inputs
int ouro_fast_layer(ouro_ctx *c, int which, int layer, int rows);          // tensor-core layer; OURO_ESTATE = not available
int ouro_fast_head(ouro_ctx *c, int which, int rows, float *logits, int32_t *argmax_dev);   // tensor-core LM head + argmax

static int forward(ouro_ctx *c, int which, int32_t *argmax_dev, float *logits_dev) {
  ModelRt &M = c->m[which];
  if (!M.present) return fail(c, OURO_ESTATE, "model not present");
  const int rows = M.blk_rows, L = M.L;
  if (rows == 0 || M.blk_L != L) return fail(c, OURO_ESTATE, "no block assembled for the current cache length");
  const ouro_model_desc &d = M.d;
  const int dt = d.dtype, dq = d.n_heads * d.head_dim, dkv = d.n_kv_heads * d.head_dim;
  cudaStream_t s = c->stream;
  Activations &a = c->a;
  ProfScope whole(c, OURO_PROF_FORWARD);
  c->cur_rows_dev = M.blk_rows_dev ? &c->st->n_rows : nullptr;
  if (ouro_fast_embed(c, which, rows) == OURO_ESTATE) {
    ProfScope ps(c, OURO_PROF_EMBED);
    launch_embed(dt, M.embed, M.blk.tok, rows, d.d_model, a.x, s);
  }
  for (int l = 0; l < d.n_layers; ++l) {
    int rc = ouro_fast_layer(c, which, l, rows);
    if (rc == OURO_OK) continue;
    if (rc != OURO_ESTATE) return rc;
    { ProfScope ps(c, OURO_PROF_NORM); launch_rmsnorm(dt, a.x, M.attn_norm[l], rows, d.d_model, d.rms_eps, a.xn, s); }
    {
      ProfScope ps(c, OURO_PROF_QKV);
      GemmSegs qkv{{M.wq[l], M.wk[l], M.wv[l]}, {dq, dkv, dkv}, 3};
      launch_gemm_simple(dt, a.xn, qkv, rows, d.d_model, a.qkv, dq + 2 * dkv, EPI_STORE, s);
    }
    { ProfScope ps(c, OURO_PROF_ROPE); launch_rope_append(d, a.qkv, M.blk.pos, M.rope_cos, M.rope_sin, rows, L, l, a.q, M.k_cache, M.v_cache, s); }
    { ProfScope ps(c, OURO_PROF_ATTENTION); launch_attention_simple(d, a.q, M.k_cache, M.v_cache, M.blk, rows, l, a.att, s); }
    {
      ProfScope ps(c, OURO_PROF_WO);
      GemmSegs wo{{M.wo[l], nullptr, nullptr}, {d.d_model, 0, 0}, 1};
      launch_gemm_simple(dt, a.att, wo, rows, dq, a.x, d.d_model, EPI_RESIDUAL, s);
    }
    { ProfScope ps(c, OURO_PROF_NORM); launch_rmsnorm(dt, a.x, M.ffn_norm[l], rows, d.d_model, d.rms_eps, a.xn, s); }
    { ProfScope ps(c, OURO_PROF_GATEUP); launch_gemm_swiglu_simple(dt, a.xn, M.w_gate[l], M.w_up[l], rows, d.d_model, d.d_ffn, a.act, s); }
    {
      ProfScope ps(c, OURO_PROF_DOWN);
      GemmSegs wd{{M.w_down[l], nullptr, nullptr}, {d.d_model, 0, 0}, 1};
      launch_gemm_simple(dt, a.act, wd, rows, d.d_ffn, a.x, d.d_model, EPI_RESIDUAL, s);
    }
  }
  int rc = ouro_fast_head(c, which, rows, logits_dev, argmax_dev);
  if (rc == OURO_ESTATE) {
    float *logits = logits_dev ? logits_dev : a.logits;
    { ProfScope ps(c, OURO_PROF_NORM); launch_rmsnorm(dt, a.x, M.final_norm, rows, d.d_model, d.rms_eps, a.xn, s); }
    {
      ProfScope ps(c, OURO_PROF_HEAD);
      GemmSegs head{{M.lm_head, nullptr, nullptr}, {d.vocab, 0, 0}, 1};
      launch_gemm_simple(dt, a.xn, head, rows, d.d_model, logits, d.vocab, EPI_STORE, s);
    }
    ProfScope pa(c, OURO_PROF_ARGMAX);
    launch_argmax(logits, rows, d.vocab, argmax_dev, s);
  } else if (rc != OURO_OK) {
    return rc;
  }
  CKL();
  return OURO_OK;
}

extern "C" int ouro_verify_forward(ouro_ctx *c, int which, int32_t *argmax_dev, float *logits_dev) {
  if (!c || which < 0 || which > 1 || !argmax_dev) return OURO_EINVAL;
  return forward(c, which, argmax_dev, logits_dev);
}

extern "C" int ouro_advance(ouro_ctx *c, int which, int32_t n) {
  if (!c || which < 0 || which > 1) return OURO_EINVAL;
  ModelRt &M = c->m[which];
  if (M.blk_rows == 0 || M.blk_is_candidate || n < 0 || n > M.blk_rows) return fail(c, OURO_ESTATE, "no causal block of that size");
  M.L += n;
  M.blk_rows = 0;
  return OURO_OK;
}

// Runs model `which` over text positions [M.L, upto) taken from seq_dev, in chunks; the outputs of the last
// chunk stay in a.argmax (row index of the last position returned through last_row).
static int feed_text(ouro_ctx *c, int which, int upto, int *last_row) {
  ModelRt &M = c->m[which];
  while (M.L < upto) {
    int n = std::min<int>(OURO_MAX_ROWS, upto - M.L);
    TRY(ouro_assemble_causal(c, which, c->seq_dev + M.L, n));
    TRY(forward(c, which, c->a.argmax, nullptr));
    M.L += n;
    M.blk_rows = 0;
    if (last_row) *last_row = n - 1;
  }
  return OURO_OK;
}

extern "C" int ouro_prefill(ouro_ctx *c, const int32_t *prompt, int32_t n) {
  if (!c || !prompt || n < 1) return OURO_EINVAL;
  ModelRt &T = c->m[OURO_TARGET];
  if (T.L != 0 || c->seq.size() != 1) return fail(c, OURO_ESTATE, "prefill needs a freshly reset context");
  if (n + 1 + c->p.gamma + c->p.K * (c->p.beta - 1) > T.d.max_seq) return fail(c, OURO_ECAPACITY, "prompt does not fit max_seq");
  for (int i = 0; i < n; ++i)
    if (prompt[i] < 0 || prompt[i] >= T.d.vocab) return fail(c, OURO_EINVAL, "prompt token out of range");
  c->seq.assign(prompt, prompt + n);
  CK(cudaMemcpyAsync(c->seq_dev, c->seq.data(), (size_t)n * 4, cudaMemcpyHostToDevice, c->stream));
  launch_set_state(c->st, c->seq_dev, n, prompt[n - 1], 0, c->stream);
  if ((c->p.flags & OURO_SEED_PROMPT) && n >= c->p.beta)
    launch_pool_update(c->pool, c->st, c->seq_dev, n - c->p.beta + 1, c->p.beta, 1, c->stream);
  CKL();
  TRY(feed_text(c, OURO_TARGET, n - 1, nullptr));
  CK(cudaStreamSynchronize(c->stream));   // c->seq must outlive the pageable upload; also surfaces launch errors
  return OURO_OK;
}

// -------------------------------------------------------------------------------------- pool
extern "C" int ouro_phrase_lookup(ouro_ctx *c, int32_t key, int32_t K, int32_t *suffix_dev, int32_t *count_dev) {
  if (!c || !suffix_dev || !count_dev || K < 0 || K > OURO_MAX_K) return OURO_EINVAL;
  launch_pool_lookup(c->pool, nullptr, 0, key, K, suffix_dev, count_dev, c->stream);
  CKL();
  return OURO_OK;
}

extern "C" int ouro_phrase_update(ouro_ctx *c, const int32_t *ngrams_dev, int32_t n) {
  if (!c || n < 0 || (n > 0 && !ngrams_dev)) return OURO_EINVAL;
  launch_pool_update(c->pool, c->st, ngrams_dev, n, c->p.beta, c->p.beta, c->stream);
  CKL();
  return OURO_OK;
}

extern "C" int ouro_pool_export(ouro_ctx *c, int32_t *ngrams, uint64_t *stamps, int32_t *n_out) {
  if (!c || !ngrams || !n_out) return OURO_EINVAL;
  const PoolDev &P = c->pool;
  size_t cap = (size_t)P.sets * P.ways;
  std::vector<int32_t> key(cap), suf(cap * std::max(1, P.S));
  std::vector<u64> stamp(cap);
  CK(cudaStreamSynchronize(c->stream));
  CK(cudaMemcpy(key.data(), P.key, cap * 4, cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(suf.data(), P.suf, suf.size() * 4, cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(stamp.data(), P.stamp, cap * 8, cudaMemcpyDeviceToHost));
  std::vector<size_t> live;
  for (size_t e = 0; e < cap; ++e) if (key[e] >= 0) live.push_back(e);
  std::sort(live.begin(), live.end(), [&](size_t a, size_t b) { return stamp[a] < stamp[b]; });
  const int beta = P.S + 1;
  for (size_t i = 0; i < live.size(); ++i) {
    size_t e = live[i];
    ngrams[i * beta] = key[e];
    for (int k = 0; k < P.S; ++k) ngrams[i * beta + 1 + k] = suf[e * P.S + k];
    if (stamps) stamps[i] = stamp[e];
  }
  *n_out = (int32_t)live.size();
  return OURO_OK;
}

extern "C" int ouro_pool_import(ouro_ctx *c, const int32_t *ngrams, int32_t n) {
  if (!c || n < 0 || (n > 0 && !ngrams)) return OURO_EINVAL;
  const int beta = c->p.beta;
  int32_t *stage = (int32_t *)c->a.logits;  // idle between forwards; [rows, vocab] floats
  size_t room = (size_t)OURO_MAX_ROWS * c->m[0].d.vocab;
  for (int done = 0; done < n;) {
    int chunk = (int)std::min<size_t>(n - done, room / beta);
    if (chunk < 1) return fail(c, OURO_ENOMEM, "no staging room for pool import");
    CK(cudaMemcpyAsync(stage, ngrams + (size_t)done * beta, (size_t)chunk * beta * 4, cudaMemcpyHostToDevice, c->stream));
    launch_pool_update(c->pool, c->st, stage, chunk, beta, beta, c->stream);
    CKL();
    CK(cudaStreamSynchronize(c->stream));
    done += chunk;
  }
  return OURO_OK;
}

// -------------------------------------------------------------------------- accept + compact
struct AcceptOut {
  int32_t A, chosen, m, n_acc;
  int32_t accepted[OURO_MAX_GAMMA + OURO_MAX_BETA];
  int32_t status;
  int32_t n_cand;     // candidates the block held (K' <= K)
};

static int accept_step(ouro_ctx *c, const int32_t *argmax_dev, AcceptOut *r) {
  ModelRt &T = c->m[OURO_TARGET];
  if (T.blk_rows == 0 || !T.blk_is_candidate || T.blk_L != T.L)
    return fail(c, OURO_ESTATE, "no verified candidate block for the current cache length");
  const int gamma = c->p.gamma, S = c->p.beta - 1, L = T.L;
  cudaStream_t s = c->stream;
  static_assert(sizeof(AcceptOut) <= PIN_INTS * 4, "pinned staging too small");
  static_assert(sizeof(AcceptOut) == (4 + OURO_MAX_GAMMA + OURO_MAX_BETA + 2) * 4 && MBOX_ACCEPT + 1 + sizeof(AcceptOut) / 4 <= MBOX_INTS,
                "acceptance record and mailbox slot disagree");
  if (c->mbox) {
    const int32_t seq = ++c->mseq;
    launch_accept_compact_harvest(T.blk, c->st, c->pool, argmax_dev, c->seq_dev, T.d, T.k_cache, T.v_cache, L, gamma, S,
                                  c->p.flags, c->mbox_dev, seq, s);
    CKL();
    TRY(mbox_wait(c, MBOX_ACCEPT, seq));
    memcpy(r, c->mbox + MBOX_ACCEPT + 1, sizeof(AcceptOut));
  } else {
    launch_accept_compact_harvest(T.blk, c->st, c->pool, argmax_dev, c->seq_dev, T.d, T.k_cache, T.v_cache, L, gamma, S,
                                  c->p.flags, nullptr, 0, s);
    CKL();
    CK(cudaMemcpyAsync(c->pin, &c->st->A, sizeof(AcceptOut), cudaMemcpyDeviceToHost, s));
    CK(cudaStreamSynchronize(s));
    memcpy(r, c->pin, sizeof(AcceptOut));
  }
  if (r->status != 0) {
    ouro_fast_mark_dirty(c);
    return fail(c, OURO_ETIMEOUT, "device status word " + std::to_string(r->status));
  }
  if (r->n_acc < 1 || r->n_acc > gamma + S + 1) return fail(c, OURO_ECUDA, "acceptance returned an impossible count");
  c->seq.insert(c->seq.end(), r->accepted, r->accepted + r->n_acc);
  T.L = L + r->n_acc;
  T.blk_rows = 0;
  ModelRt &D = c->m[OURO_DRAFT];
  if (D.present) D.L = std::min(D.L, L + std::min(r->A + 1, gamma));   // draft cache keeps the accepted prefix only
  c->step += 1;
  return OURO_OK;
}

extern "C" int ouro_accept_and_compact(ouro_ctx *c, const int32_t *argmax_dev, int32_t *n_acc, int32_t *chosen,
                                       int32_t *accurate, int32_t *accepted) {
  if (!c || !argmax_dev) return OURO_EINVAL;
  AcceptOut r;
  TRY(accept_step(c, argmax_dev, &r));
  if (n_acc) *n_acc = r.n_acc;
  if (chosen) *chosen = r.chosen;
  if (accurate) *accurate = r.A;
  if (accepted) memcpy(accepted, r.accepted, (size_t)r.n_acc * 4);
  return OURO_OK;
}

// One verification step in one call: lookup + packing, the target forward, acceptance + compaction + harvest.
extern "C" int ouro_verify_step(ouro_ctx *c, const int32_t *draft_dev, int32_t *n_acc, int32_t *chosen, int32_t *accurate,
                                int32_t *accepted) {
  if (!c || !draft_dev) return OURO_EINVAL;
  TRY(ouro_assemble_candidates(c, draft_dev, nullptr, nullptr));
  TRY(forward(c, OURO_TARGET, c->a.argmax, nullptr));
  return ouro_accept_and_compact(c, c->a.argmax, n_acc, chosen, accurate, accepted);
}

// ------------------------------------------------------------------------------------- draft
// Eq. 1.  The draft model first catches up on the text it has not cached (including the pending token),
// which yields d_1; each further token costs one single-row forward.  With an external drafter the
// tokens come from the callback; a present draft model still runs the same forwards on them, so that
// replayed drafts cost what real drafting costs.
// Section 3.1 (see ouro_draft in the header): the draft model drafts phrase by phrase.  Every round is one draft
// forward over the text it has not cached yet plus the pool phrases that start with the last known token, and
// yields one token plus the matched phrase prefix.  Two small reads per round tell the host the block's row
// count and how far the draft and its cache advanced.
static int draft_step_phrases(ouro_ctx *c, int32_t *out_dev, int *calls) {
  const int gamma = c->p.gamma, S = c->p.beta - 1, K = c->p.K;
  ModelRt &D = c->m[OURO_DRAFT];
  cudaStream_t s = c->stream;
  const int n_seq = (int)c->seq.size();
  if (n_seq + gamma + K * S > D.d.max_seq) return fail(c, OURO_ECAPACITY, "draft cache full");
  // text that does not fit the first round's block beside the candidates goes through plain causal blocks
  if (n_seq - D.L + K * S > OURO_MAX_ROWS) TRY(feed_text(c, OURO_DRAFT, n_seq - 1, nullptr));
  int have = 0;
  while (have < gamma) {
    const int n = have == 0 ? n_seq - D.L : 1;
    const int32_t *tokens = have == 0 ? c->seq_dev + D.L : out_dev + have - 1;
    if (n < 1) return fail(c, OURO_ESTATE, "draft cache ahead of the text");
    launch_draft_lookup_assemble(c->pool, D.blk, c->st, tokens, n, c->cand_suffix, c->cand_count, D.L, S, K, s);
    CKL();
    CK(cudaMemcpyAsync(c->pin, &c->st->n_rows, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    CK(cudaStreamSynchronize(s));
    D.blk_rows = c->pin[0];
    D.blk_rows_dev = false;
    D.blk_L = D.L;
    D.blk_is_candidate = true;
    if (D.blk_rows < n || D.blk_rows > n + K * S) return fail(c, OURO_ECUDA, "draft block has an impossible row count");
    TRY(forward(c, OURO_DRAFT, c->a.argmax, nullptr));
    launch_draft_accept_compact(D.blk, c->st, c->a.argmax, out_dev, have, gamma, D.d, D.k_cache, D.v_cache, D.L, n, S, s);
    CKL();
    CK(cudaMemcpyAsync(c->pin, &c->st->d_keep, 2 * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    CK(cudaStreamSynchronize(s));
    const int keep = c->pin[0], cached = c->pin[1];
    if (keep < 1 || keep > gamma - have || cached < 0 || cached > keep)
      return fail(c, OURO_ECUDA, "drafting round returned an impossible count");
    D.L += n + cached;
    D.blk_rows = 0;
    have += keep;
    *calls += 1;
  }
  return OURO_OK;
}

static int draft_step(ouro_ctx *c, int32_t *out_dev, int *calls) {
  const int gamma = c->p.gamma;
  ModelRt &D = c->m[OURO_DRAFT];
  const bool ext = c->drafter != nullptr;
  if (!ext && !D.present) return fail(c, OURO_ESTATE, "neither a draft model nor an external drafter");
  if (ext) {
    int32_t tmp[OURO_MAX_GAMMA];
    if (c->drafter(c->drafter_user, c->seq.data(), (int32_t)c->seq.size(), gamma, c->step, tmp) != 0)
      return fail(c, OURO_EINVAL, "external drafter failed");
    for (int i = 0; i < gamma; ++i)
      if (tmp[i] < 0 || tmp[i] >= c->m[0].d.vocab) return fail(c, OURO_EINVAL, "external drafter returned a token out of range");
    memcpy(c->pin, tmp, (size_t)gamma * 4);
    CK(cudaMemcpyAsync(out_dev, c->pin, (size_t)gamma * 4, cudaMemcpyHostToDevice, c->stream));
    CK(cudaStreamSynchronize(c->stream));   // the pinned staging is reused by later calls
  }
  if (!D.present) return OURO_OK;
  if (!ext && (c->p.flags & OURO_DRAFT_PHRASES)) return draft_step_phrases(c, out_dev, calls);
  if ((int)c->seq.size() + gamma + c->p.window > D.d.max_seq) return fail(c, OURO_ECAPACITY, "draft cache full");
  if (c->p.window > 0) {
    // Section 3.1, phrase generation during drafting (see ouro_draft in the header): every draft forward carries the
    // lookahead window behind its text rows; its outputs refill the window and feed the pool, all on the device.
    const int W = c->p.window, n_seq = (int)c->seq.size();
    if (n_seq - D.L + W > OURO_MAX_ROWS) TRY(feed_text(c, OURO_DRAFT, n_seq - 1, nullptr));
    for (int i = 0; i < gamma; ++i) {
      const int n = i == 0 ? n_seq - D.L : 1;
      if (n < 1) return fail(c, OURO_ESTATE, "draft cache ahead of the text");
      launch_draft_window_assemble(D.blk, c->st, i == 0 ? c->seq_dev + D.L : out_dev + i - 1, n, c->win_dev, W, c->seq_dev,
                                   D.L, c->stream);
      D.blk_rows = n + W;
      D.blk_rows_dev = false;
      D.blk_L = D.L;
      D.blk_is_candidate = true;
      TRY(forward(c, OURO_DRAFT, c->a.argmax, nullptr));
      launch_draft_window_harvest(D.blk, c->st, c->pool, c->a.argmax, ext ? nullptr : out_dev + i, n, W, c->win_dev, c->stream);
      D.L += n;
      D.blk_rows = 0;
      *calls += 1;
    }
    CKL();
    return OURO_OK;
  }
  int last = 0;
  TRY(feed_text(c, OURO_DRAFT, (int)c->seq.size(), &last));
  *calls += 1;
  if (!ext) launch_pick_token(c->a.argmax, last, out_dev, c->stream);
  for (int i = 1; i < gamma; ++i) {
    TRY(ouro_assemble_causal(c, OURO_DRAFT, out_dev + i - 1, 1));
    TRY(forward(c, OURO_DRAFT, c->a.argmax, nullptr));
    D.L += 1;
    D.blk_rows = 0;
    *calls += 1;
    if (!ext) launch_pick_token(c->a.argmax, 0, out_dev + i, c->stream);
  }
  CKL();
  return OURO_OK;
}

extern "C" int ouro_draft(ouro_ctx *c, int32_t *draft_dev) {
  if (!c || !draft_dev) return OURO_EINVAL;
  int calls = 0;
  return draft_step(c, draft_dev, &calls);
}

// ------------------------------------------------------------------------------------- loops
extern "C" int ouro_generate(ouro_ctx *c, const int32_t *prompt, int32_t n_prompt, int32_t max_new, int32_t keep_pool,
                             int32_t *out, int32_t *n_out, ouro_stats *stats) {
  if (!c || !prompt || !out || !n_out || max_new < 0) return OURO_EINVAL;
  TRY(ouro_reset(c, keep_pool));
  TRY(ouro_prefill(c, prompt, n_prompt));
  ouro_stats st{};
  ModelRt &T = c->m[OURO_TARGET];
  const int gamma = c->p.gamma, S = c->p.beta - 1;
  cudaStream_t s = c->stream;
  CK(cudaEventRecord(c->ev[0], s));
  int n = 0;
  bool stop = false;
  while (n < max_new && !stop) {
    if (T.L + 1 + gamma + c->p.K * S > T.d.max_seq) return fail(c, OURO_ECAPACITY, "target cache full");
    CK(cudaEventRecord(c->ev[1], s));
    TRY(draft_step(c, c->draft_dev, &st.draft_calls));
    CK(cudaEventRecord(c->ev[2], s));
    TRY(ouro_assemble_candidates(c, c->draft_dev, nullptr, nullptr));
    CK(cudaEventRecord(c->ev[3], s));
    TRY(forward(c, OURO_TARGET, c->a.argmax, nullptr));
    CK(cudaEventRecord(c->ev[4], s));
    AcceptOut r;
    TRY(accept_step(c, c->a.argmax, &r));
    float ms = 0.f;
    CK(cudaEventSynchronize(c->ev[4]));               // reached long ago; makes the runtime see it as complete
    CK(cudaEventElapsedTime(&ms, c->ev[1], c->ev[2]));
    st.ms_draft += ms;
    CK(cudaEventElapsedTime(&ms, c->ev[3], c->ev[4]));
    st.ms_target += ms;
    st.target_calls += 1;
    st.full_accepts += r.A == gamma;
    st.suffix_tokens += r.chosen >= 0 ? r.m : 0;
    st.candidates += r.n_cand;
    for (int i = 0; i < r.n_acc && n < max_new; ++i) {
      out[n++] = r.accepted[i];
      if (c->p.eos_token >= 0 && r.accepted[i] == c->p.eos_token) { stop = true; break; }
    }
  }
  CK(cudaEventRecord(c->ev[5], s));
  CK(cudaEventSynchronize(c->ev[5]));
  CK(cudaEventElapsedTime(&st.ms_total, c->ev[0], c->ev[5]));
  st.n_tokens = n;
  *n_out = n;
  if (stats) *stats = st;
  return OURO_OK;
}

extern "C" int ouro_generate_vanilla(ouro_ctx *c, const int32_t *prompt, int32_t n_prompt, int32_t max_new, int32_t *out,
                                     int32_t *n_out, ouro_stats *stats) {
  if (!c || !prompt || !out || !n_out || max_new < 0) return OURO_EINVAL;
  TRY(ouro_reset(c, 1));
  const uint32_t flags = c->p.flags;
  c->p.flags &= ~(uint32_t)OURO_SEED_PROMPT;            // plain decoding leaves the pool alone
  int rc = ouro_prefill(c, prompt, n_prompt);
  c->p.flags = flags;
  if (rc != OURO_OK) return rc;
  ouro_stats st{};
  ModelRt &T = c->m[OURO_TARGET];
  cudaStream_t s = c->stream;
  if (T.L + max_new > T.d.max_seq) return fail(c, OURO_ECAPACITY, "target cache too small for max_new tokens");
  const int base = (int)c->seq.size();
  CK(cudaEventRecord(c->ev[0], s));
  int n = 0;
  const bool has_eos = c->p.eos_token >= 0;
  while (n < max_new) {
    TRY(ouro_assemble_causal(c, OURO_TARGET, &c->st->pending, 1));
    TRY(forward(c, OURO_TARGET, c->a.argmax, nullptr));
    launch_vanilla_accept(c->st, c->a.argmax, c->seq_dev, s);
    CKL();
    T.L += 1;
    T.blk_rows = 0;
    st.target_calls += 1;
    n += 1;
    if (has_eos) {   // the stop token must be seen on the host before the next forward
      CK(cudaMemcpyAsync(c->pin, &c->st->pending, 4, cudaMemcpyDeviceToHost, s));
      CK(cudaStreamSynchronize(s));
      if (c->pin[0] == c->p.eos_token) break;
    }
  }
  CK(cudaEventRecord(c->ev[5], s));
  CK(cudaMemcpyAsync(out, c->seq_dev + base, (size_t)n * 4, cudaMemcpyDeviceToHost, s));
  CK(cudaMemcpyAsync(c->pin, &c->st->status, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  CK(cudaStreamSynchronize(s));
  if (c->pin[0] != 0) {
    ouro_fast_mark_dirty(c);
    return fail(c, OURO_ETIMEOUT, "device status word " + std::to_string(c->pin[0]));
  }
  CK(cudaEventElapsedTime(&st.ms_total, c->ev[0], c->ev[5]));
  st.ms_target = st.ms_total;
  c->seq.insert(c->seq.end(), out, out + n);
  st.n_tokens = n;
  *n_out = n;
  if (stats) *stats = st;
  return OURO_OK;
}
