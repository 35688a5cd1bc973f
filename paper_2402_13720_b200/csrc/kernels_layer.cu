// Layer kernels, generic versions: embedding gather, RMSNorm, rotary + cache append, plain GEMMs and the
// candidate-masked attention in their simplest correct form (any shape, fp32 or bf16 storage, fp32
// arithmetic).  They serve the small fp32 configuration and shapes the tensor-core kernels do not take.
//
// Design rule shared by every kernel here and by their fast counterparts: the value computed for the
// token at absolute position P depends only on that token's own row and on the keys it may see, taken
// in ascending position order in fixed groups.  It never depends on how many other rows the block has.
// That is what makes Ouroboros output bit-identical to one-token-at-a-time greedy decoding on this
// library (the paper observes small differences "caused by floating point error", Appendix A).
#include "ouro_internal.h"

#define FULL 0xffffffffu

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T> struct Vec;       // 16-byte vector of T
template <> struct Vec<float> {
  static constexpr int N = 4;
  float4 v;
  __device__ __forceinline__ void load(const float *p) { v = *reinterpret_cast<const float4 *>(p); }
  __device__ __forceinline__ float get(int i) const { return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w; }
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  uint4 v;
  __device__ __forceinline__ void load(const __nv_bfloat16 *p) { v = *reinterpret_cast<const uint4 *>(p); }
  __device__ __forceinline__ float get(int i) const {
    uint32_t w = (i >> 1) == 0 ? v.x : (i >> 1) == 1 ? v.y : (i >> 1) == 2 ? v.z : v.w;
    return __uint_as_float((i & 1) ? (w & 0xffff0000u) : (w << 16));
  }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(FULL, v, o));
  return v;
}

// ------------------------------------------------------------------------------ rotary table
// cos/sin of pos * theta^(-2i/h), evaluated in double once at set-up.
__global__ void rope_table_kernel(float *cos_t, float *sin_t, int max_seq, int half, double theta) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= max_seq * half) return;
  int pos = idx / half, i = idx % half;
  double ang = (double)pos * pow(theta, -(double)i / (double)half);
  cos_t[idx] = (float)cos(ang);
  sin_t[idx] = (float)sin(ang);
}
void launch_rope_table(float *cos_t, float *sin_t, int max_seq, int head_dim, float theta, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  int n = max_seq * (head_dim / 2);
  rope_table_kernel<<<(n + 255) / 256, 256, 0, s>>>(cos_t, sin_t, max_seq, head_dim / 2, (double)theta);
}

// --------------------------------------------------------------------------------- embedding
template <typename T>
__global__ void embed_kernel(const T *E, const int32_t *tok, int d, float *x) {
  pdl_trigger();
  pdl_wait();
  const T *src = E + (size_t)tok[blockIdx.x] * d;
  float *dst = x + (size_t)blockIdx.x * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) dst[i] = to_f<T>(src[i]);
}
void launch_embed(int dtype, const void *E, const int32_t *tok, int rows, int d, float *x, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  if (dtype == OURO_BF16) launch_pdl(embed_kernel<__nv_bfloat16>, rows, 256, 0, s, (const __nv_bfloat16 *)E, tok, d, x);
  else launch_pdl(embed_kernel<float>, rows, 256, 0, s, (const float *)E, tok, d, x);
}

// ----------------------------------------------------------------------------------- RMSNorm
// out = g * x / sqrt(mean(x^2) + eps); one block per row, fixed reduction order.
template <typename T>
__global__ void rmsnorm_kernel(const float *x, const T *g, int d, float eps, T *out) {
  pdl_trigger();
  pdl_wait();
  const float *row = x + (size_t)blockIdx.x * d;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) ss += row[i] * row[i];
  __shared__ float part[32];
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += part[w];
  float inv = 1.0f / sqrtf(tot / (float)d + eps);
  T *o = out + (size_t)blockIdx.x * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) o[i] = from_f<T>(to_f<T>(g[i]) * (row[i] * inv));
}
void launch_rmsnorm(int dtype, const float *x, const void *g, int rows, int d, float eps, void *out, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  if (dtype == OURO_BF16)
    launch_pdl(rmsnorm_kernel<__nv_bfloat16>, rows, 256, 0, s, x, (const __nv_bfloat16 *)g, d, eps, (__nv_bfloat16 *)out);
  else launch_pdl(rmsnorm_kernel<float>, rows, 256, 0, s, x, (const float *)g, d, eps, (float *)out);
}

// -------------------------------------------------------------------------------- plain GEMM
// Y[r, n] (+)= sum_k X[r, k] * W[n, k].  One warp per output column, lanes stride over k in 16-byte
// vectors, rows in register tiles of RT.  The k order per output element is fixed by (lane, K) alone.
template <typename T, int RT>
__device__ __forceinline__ void warp_dot_rows(const T *X, const T *wrow, int r0, int rows, int K, float *acc) {
  constexpr int V = Vec<T>::N;
  int lane = threadIdx.x & 31;
#pragma unroll
  for (int i = 0; i < RT; ++i) acc[i] = 0.f;
  for (int k = lane * V; k < K; k += 32 * V) {
    Vec<T> w;
    w.load(wrow + k);
#pragma unroll
    for (int i = 0; i < RT; ++i) {
      if (r0 + i < rows) {
        Vec<T> xv;
        xv.load(X + (size_t)(r0 + i) * K + k);
#pragma unroll
        for (int e = 0; e < V; ++e) acc[i] = fmaf(xv.get(e), w.get(e), acc[i]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < RT; ++i) acc[i] = warp_sum(acc[i]);
}

template <typename T>
__global__ void gemm_simple_kernel(const T *X, GemmSegs W, int rows, int K, float *Y, int ldy, int epi) {
  int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int ntot = W.n[0] + (W.count > 1 ? W.n[1] : 0) + (W.count > 2 ? W.n[2] : 0);
  if (n >= ntot) return;
  int seg = 0, nl = n;
  while (nl >= W.n[seg]) nl -= W.n[seg++];
  const T *wrow = (const T *)W.w[seg] + (size_t)nl * K;
  constexpr int RT = 8;
  float acc[RT];
  for (int r0 = 0; r0 < rows; r0 += RT) {
    warp_dot_rows<T, RT>(X, wrow, r0, rows, K, acc);
    if ((threadIdx.x & 31) == 0) {
#pragma unroll
      for (int i = 0; i < RT; ++i)
        if (r0 + i < rows) {
          float *y = Y + (size_t)(r0 + i) * ldy + n;
          *y = epi == EPI_RESIDUAL ? *y + acc[i] : acc[i];
        }
    }
  }
}
void launch_gemm_simple(int dtype, const void *X, const GemmSegs &W, int rows, int K, float *Y, int ldy, int epi,
                        cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  int ntot = 0;
  for (int i = 0; i < W.count; ++i) ntot += W.n[i];
  int grid = (ntot + 3) / 4;
  if (dtype == OURO_BF16) gemm_simple_kernel<__nv_bfloat16><<<grid, 128, 0, s>>>((const __nv_bfloat16 *)X, W, rows, K, Y, ldy, epi);
  else gemm_simple_kernel<float><<<grid, 128, 0, s>>>((const float *)X, W, rows, K, Y, ldy, epi);
}

// act[r, n] = SiLU(X Wg^T)[r, n] * (X Wu^T)[r, n]
template <typename T>
__global__ void gemm_swiglu_simple_kernel(const T *X, const T *Wg, const T *Wu, int rows, int K, int F, T *act) {
  int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (n >= F) return;
  constexpr int RT = 8;
  float g[RT], u[RT];
  for (int r0 = 0; r0 < rows; r0 += RT) {
    warp_dot_rows<T, RT>(X, Wg + (size_t)n * K, r0, rows, K, g);
    warp_dot_rows<T, RT>(X, Wu + (size_t)n * K, r0, rows, K, u);
    if ((threadIdx.x & 31) == 0) {
#pragma unroll
      for (int i = 0; i < RT; ++i)
        if (r0 + i < rows) act[(size_t)(r0 + i) * F + n] = from_f<T>(g[i] / (1.0f + expf(-g[i])) * u[i]);
    }
  }
}
void launch_gemm_swiglu_simple(int dtype, const void *X, const void *Wg, const void *Wu, int rows, int K, int F,
                               void *act, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  int grid = (F + 3) / 4;
  if (dtype == OURO_BF16)
    gemm_swiglu_simple_kernel<__nv_bfloat16><<<grid, 128, 0, s>>>((const __nv_bfloat16 *)X, (const __nv_bfloat16 *)Wg,
                                                                  (const __nv_bfloat16 *)Wu, rows, K, F, (__nv_bfloat16 *)act);
  else
    gemm_swiglu_simple_kernel<float><<<grid, 128, 0, s>>>((const float *)X, (const float *)Wg, (const float *)Wu, rows, K, F,
                                                          (float *)act);
}

// ------------------------------------------------------------------- rotary + cache append
// q and k head vectors: pairs (i, i + h/2) rotated by the row's position; k and v of row r go to cache
// slot L + r of this layer.
template <typename T>
__global__ void rope_append_kernel(const float *qkv, const int32_t *pos, const float *cos_t, const float *sin_t,
                                   int H, int Hkv, int h, int L, size_t layer_off, T *q, T *k_cache, T *v_cache) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x, half = h >> 1, dq = H * h, dkv = Hkv * h;
  const float *row = qkv + (size_t)r * (dq + 2 * dkv);
  const float *c = cos_t + (size_t)pos[r] * half, *s = sin_t + (size_t)pos[r] * half;
  for (int idx = threadIdx.x; idx < (H + Hkv) * half; idx += blockDim.x) {
    int head = idx / half, i = idx % half;
    const float *src = head < H ? row + head * h : row + dq + (head - H) * h;
    float a = src[i], b = src[i + half];
    float ra = a * c[i] - b * s[i], rb = b * c[i] + a * s[i];
    T *dst = head < H ? q + (size_t)r * dq + head * h : k_cache + layer_off + (size_t)(L + r) * dkv + (head - H) * h;
    dst[i] = from_f<T>(ra);
    dst[i + half] = from_f<T>(rb);
  }
  for (int i = threadIdx.x; i < dkv; i += blockDim.x)
    v_cache[layer_off + (size_t)(L + r) * dkv + i] = from_f<T>(row[dq + dkv + i]);
}
void launch_rope_append(const ouro_model_desc &d, const float *qkv, const int32_t *pos, const float *cos_t,
                        const float *sin_t, int rows, int L, int layer, void *q, void *k_cache, void *v_cache,
                        cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  size_t off = (size_t)layer * d.max_seq * d.n_kv_heads * d.head_dim;
  if (d.dtype == OURO_BF16)
    launch_pdl(rope_append_kernel<__nv_bfloat16>, rows, 256, 0, s, qkv, pos, cos_t, sin_t, (int)d.n_heads, (int)d.n_kv_heads,
               (int)d.head_dim, L, off, (__nv_bfloat16 *)q, (__nv_bfloat16 *)k_cache, (__nv_bfloat16 *)v_cache);
  else
    launch_pdl(rope_append_kernel<float>, rows, 256, 0, s, qkv, pos, cos_t, sin_t, (int)d.n_heads, (int)d.n_kv_heads,
               (int)d.head_dim, L, off, (float *)q, (float *)k_cache, (float *)v_cache);
}

// ------------------------------------------------------------ candidate-masked attention (plain)
// One warp per (row, head).  Keys are visited by virtual position p = 0 .. n_vis-1 in groups of 32 (lane
// = p mod 32), mapped to cache slots by the row's two ranges, so a suffix token sees the same key order
// it would see in plain decoding.  Online softmax across groups in ascending order.
template <typename T>
__global__ void attention_simple_kernel(const T *q, const T *k_cache, const T *v_cache, BlockDev b, int H, int Hkv,
                                        int h, size_t layer_off, float scale, T *out) {
  extern __shared__ float sq[];  // [warps][h]
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int r = blockIdx.x, a = blockIdx.y * (blockDim.x >> 5) + warp;
  if (a >= H) return;
  int kvh = a / (H / Hkv), dkv = Hkv * h;
  float *myq = sq + warp * h;
  for (int i = lane; i < h; i += 32) myq[i] = to_f<T>(q[(size_t)r * H * h + a * h + i]);
  __syncwarp();
  int lin_end = b.lin_end[r], seg_start = b.seg_start[r], n_vis = lin_end + b.seg_len[r];
  const T *kb = k_cache + layer_off + kvh * h, *vb = v_cache + layer_off + kvh * h;
  float m = -INFINITY, l = 0.f;
  float o[4] = {0.f, 0.f, 0.f, 0.f};  // dims lane, lane+32, .. (h <= 128)
  int nd = h >> 5;
  for (int p0 = 0; p0 < n_vis; p0 += 32) {
    int p = p0 + lane;
    bool valid = p < n_vis;
    int slot = p < lin_end ? p : seg_start + (p - lin_end);
    float sc = -INFINITY;
    if (valid) {
      const T *kr = kb + (size_t)slot * dkv;
      float acc = 0.f;
      for (int i = 0; i < h; i += Vec<T>::N) {
        Vec<T> kv;
        kv.load(kr + i);
#pragma unroll
        for (int e = 0; e < Vec<T>::N; ++e) acc = fmaf(myq[i + e], kv.get(e), acc);
      }
      sc = acc * scale;
    }
    float m_new = fmaxf(m, warp_max(sc));
    float corr = expf(m - m_new);
    float pw = valid ? expf(sc - m_new) : 0.f;
    l = l * corr + warp_sum(pw);
#pragma unroll
    for (int dd = 0; dd < 4; ++dd) o[dd] *= corr;
    int cnt = min(32, n_vis - p0);
    for (int t = 0; t < cnt; ++t) {
      float pt = __shfl_sync(FULL, pw, t);
      int st = __shfl_sync(FULL, slot, t);
      const T *vr = vb + (size_t)st * dkv;
#pragma unroll
      for (int dd = 0; dd < 4; ++dd)
        if (dd < nd) o[dd] = fmaf(pt, to_f<T>(vr[lane + 32 * dd]), o[dd]);
    }
    m = m_new;
  }
  float inv = 1.0f / l;
#pragma unroll
  for (int dd = 0; dd < 4; ++dd)
    if (dd < nd) out[(size_t)r * H * h + a * h + lane + 32 * dd] = from_f<T>(o[dd] * inv);
}
void launch_attention_simple(const ouro_model_desc &d, const void *q, const void *k_cache, const void *v_cache,
                             const BlockDev &b, int rows, int layer, void *out, cudaStream_t s) {
  OURO_COUNT_LAUNCH();
  size_t off = (size_t)layer * d.max_seq * d.n_kv_heads * d.head_dim;
  int warps = 4;
  dim3 grid(rows, (d.n_heads + warps - 1) / warps);
  size_t smem = (size_t)warps * d.head_dim * sizeof(float);
  float scale = 1.0f / sqrtf((float)d.head_dim);
  if (d.dtype == OURO_BF16)
    attention_simple_kernel<__nv_bfloat16><<<grid, warps * 32, smem, s>>>((const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k_cache,
                                                                          (const __nv_bfloat16 *)v_cache, b, d.n_heads, d.n_kv_heads,
                                                                          d.head_dim, off, scale, (__nv_bfloat16 *)out);
  else
    attention_simple_kernel<float><<<grid, warps * 32, smem, s>>>((const float *)q, (const float *)k_cache, (const float *)v_cache, b,
                                                                  d.n_heads, d.n_kv_heads, d.head_dim, off, scale, (float *)out);
}
