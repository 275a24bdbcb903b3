// Memory-bound pieces of the probes: row RMS statistics, the last-token query (Algorithm 1,
// "q <- X_N W_Q"), the head-mean softmax of Eq. 4, the score fusion of Eq. 13-14, the rotary
// table, the RMSNorm-gain fold and the first-token head.  fp32 arithmetic throughout.
#include "spts_common.cuh"

namespace spts {

namespace {

template <typename T> struct Vec16;
template <> struct Vec16<float> { static constexpr int N = 4; };
template <> struct Vec16<bf16> { static constexpr int N = 8; };

template <typename T>
__device__ __forceinline__ void load16(const T* p, float* out);
template <>
__device__ __forceinline__ void load16<float>(const float* p, float* out) {
  float4 v = *reinterpret_cast<const float4*>(p);
  out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
template <>
__device__ __forceinline__ void load16<bf16>(const bf16* p, float* out) {
  uint4 v = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out[2 * i] = __uint_as_float(w[i] << 16);
    out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

// rstd[n] = 1 / sqrt(mean(x_n^2) + eps); one warp per row.
// With a row list (idx != nullptr) only the N listed rows are recomputed: the rows a block did not update keep the
// statistic they had.
template <typename T>
__global__ void rstd_kernel(const T* __restrict__ X, const int32_t* __restrict__ idx, int N, int D, float eps,
                            float* __restrict__ rstd) {
  constexpr int V = Vec16<T>::N;
  int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= N) return;
  if (idx != nullptr) row = idx[row];
  int lane = threadIdx.x & 31;
  const T* x = X + (size_t)row * D;
  float s = 0.f;
  for (int c = lane * V; c < D; c += 32 * V) {
    float v[V];
    load16<T>(x + c, v);
#pragma unroll
    for (int i = 0; i < V; ++i) s = fmaf(v[i], v[i], s);
  }
  s = warp_sum(s);
  if (lane == 0) rstd[row] = 1.0f / sqrtf(s / (float)D + eps);
}

// cos/sin table for rotary embedding: cs[n, i] = (cos, sin)(pos[n] * theta^(-2i/d)), angles in fp64.
__global__ void rope_table_kernel(const int32_t* __restrict__ pos, int N, int half, double theta,
                                  float2* __restrict__ cs) {
  size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= (size_t)N * half) return;
  int n = (int)(t / half), i = (int)(t - (size_t)n * half);
  double inv = exp2(-(double)(2 * i) / (double)(2 * half) * log2(theta));
  double a = (double)pos[n] * inv;
  double s, c;
  sincos(a, &s, &c);
  cs[t] = make_float2((float)c, (float)s);
}

// q[h, :] = RoPE(rstd * x_last . Wq[h*d + :, :]); one warp per rotary pair (j, j + d/2).
// With `last_rows` (packed batch) block row y serves sequence y: x, rstd_last and cs_last then point at row 0 of the
// packed arrays and the sequence's last row is looked up; q gets HD floats per sequence.
template <typename T>
__global__ void q_last_kernel(const T* __restrict__ x, const T* __restrict__ wq, int D, int d, int HD,
                              float rs_scale_dummy, const float* __restrict__ rstd_last,
                              const float2* __restrict__ cs_last, float* __restrict__ q,
                              const int32_t* __restrict__ seq_start) {
  constexpr int V = Vec16<T>::N;
  int pair = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int half = d >> 1;
  if (pair >= HD / 2) return;
  if (seq_start != nullptr) {
    const int last = seq_start[blockIdx.y + 1] - 1;
    x += (size_t)last * D;
    rstd_last += last;
    cs_last += (size_t)last * half;
    q += (size_t)blockIdx.y * HD;
  }
  int lane = threadIdx.x & 31;
  int h = pair / half, i = pair - h * half;
  const T* w1 = wq + (size_t)(h * d + i) * D;
  const T* w2 = wq + (size_t)(h * d + i + half) * D;
  float a1 = 0.f, a2 = 0.f;
  for (int c = lane * V; c < D; c += 32 * V) {
    float xv[V], u[V], v[V];
    load16<T>(x + c, xv);
    load16<T>(w1 + c, u);
    load16<T>(w2 + c, v);
#pragma unroll
    for (int e = 0; e < V; ++e) { a1 = fmaf(xv[e], u[e], a1); a2 = fmaf(xv[e], v[e], a2); }
  }
  a1 = warp_sum(a1);
  a2 = warp_sum(a2);
  if (lane == 0) {
    float rs = *rstd_last;
    a1 *= rs; a2 *= rs;
    float2 c = cs_last[i];
    q[h * d + i] = a1 * c.x - a2 * c.y;
    q[h * d + i + half] = a2 * c.x + a1 * c.y;
  }
}

// per-head max and sum of exp over the N logits of one head
// Row r of the logits belongs to query (r % (w * G)) / G of a window of the last w candidates (w = 1: the last
// token only); that query sees the keys n < N - w + 1 + query (causal).  `scale` multiplies the raw logits.
__device__ __forceinline__ int pap_row_keys(int r, int N, int w, int G) { return N - w + 1 + (r % (w * G)) / G; }

// max and sum of exp of l[0..N) * scale -> out[0], out[1]; the whole block takes part
__device__ __forceinline__ void head_stats_body(const float* __restrict__ l, int N, float scale, float* __restrict__ out) {
  __shared__ float red[32];
  __shared__ float bcast;
  int tid = threadIdx.x;
  float m = -INFINITY;
  for (int n = tid; n < N; n += blockDim.x) m = fmaxf(m, l[n] * scale);
  m = warp_max(m);
  if ((tid & 31) == 0) red[tid >> 5] = m;
  __syncthreads();
  if (tid < 32) {
    float v = tid < (blockDim.x >> 5) ? red[tid] : -INFINITY;
    v = warp_max(v);
    if (tid == 0) bcast = v;
  }
  __syncthreads();
  m = bcast;
  float s = 0.f;
  for (int n = tid; n < N; n += blockDim.x) s += expf(l[n] * scale - m);
  s = warp_sum(s);
  __syncthreads();
  if ((tid & 31) == 0) red[tid >> 5] = s;
  __syncthreads();
  if (tid < 32) {
    float v = tid < (blockDim.x >> 5) ? red[tid] : 0.f;
    v = warp_sum(v);
    if (tid == 0) { out[0] = m; out[1] = v; }
  }
}

__global__ void __launch_bounds__(1024)
pap_head_stats_kernel(const float* __restrict__ logits, int ld, int N_all, int w, int G, float scale,
                      float* __restrict__ stats) {
  head_stats_body(logits + (size_t)blockIdx.x * ld, pap_row_keys(blockIdx.x, N_all, w, G), scale, stats + 2 * blockIdx.x);
}

// Packed batch: block (h, b) takes head h over the rows of sequence b; stats [n_seq][H][2].  The same reduction, thread
// for thread, as the single-sequence kernel runs on that sequence alone.
__global__ void __launch_bounds__(1024)
pap_head_stats_batch_kernel(const float* __restrict__ logits, int ld, const int32_t* __restrict__ seq_start,
                            float* __restrict__ stats) {
  const int s0 = seq_start[blockIdx.y];
  head_stats_body(logits + (size_t)blockIdx.x * ld + s0, seq_start[blockIdx.y + 1] - s0, 1.0f,
                  stats + 2 * ((size_t)blockIdx.y * gridDim.x + blockIdx.x));
}

// S[n] = (1/H) sum_h exp(l[h, n] - max_{b,h}) / sum_{b,h} with b the sequence of row n (Eq. 4 per prompt)
__global__ void pap_mean_batch_kernel(const float* __restrict__ logits, int ld, int total, int H,
                                      const int32_t* __restrict__ row_seq, const float* __restrict__ stats,
                                      float* __restrict__ S) {
  int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= total) return;
  const float* st = stats + 2 * (size_t)row_seq[n] * H;
  float acc = 0.f;
  for (int r = 0; r < H; ++r) acc += expf(logits[(size_t)r * ld + n] * 1.0f - st[2 * r]) / st[2 * r + 1];
  S[n] = acc * (1.0f / (float)H);
}

// row_seq[n] = the sequence that owns packed row n (seq_start ascending, n_seq + 1 entries)
__global__ void batch_row_seq_kernel(const int32_t* __restrict__ seq_start, int n_seq, int total, int32_t* __restrict__ row_seq) {
  int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= total) return;
  int lo = 0, hi = n_seq;                     // seq_start[lo] <= n < seq_start[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (seq_start[mid] <= n) lo = mid; else hi = mid;
  }
  row_seq[n] = lo;
}

// vt_col[a] = column of the transposed V copy that active row a goes to: sequence b's columns start at vt0[b] (a
// multiple of 8, so that a TMA box of that sequence starts on a 16-byte boundary)
__global__ void batch_vt_col_kernel(const int32_t* __restrict__ act_off, const int32_t* __restrict__ vt0, int n_seq,
                                    int n_act, int32_t* __restrict__ vt_col) {
  int a = blockIdx.x * blockDim.x + threadIdx.x;
  if (a >= n_act) return;
  int lo = 0, hi = n_seq;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (act_off[mid] <= a) lo = mid; else hi = mid;
  }
  vt_col[a] = vt0[lo] + (a - act_off[lo]);
}

// The selected rows of every sequence go to that sequence's cache: K^ = K[T_a] and the positions by the (global)
// index list, V^ from the packed projection output.  Active row a of the batch belongs to the sequence b with
// act_off[b] <= a < act_off[b + 1] and is that cache's row a - act_off[b].  16 bytes per thread.
struct BatchCachePtrs { void* const* k; void* const* v; int32_t* const* pos; };
__global__ void batch_cache_fill_kernel(const uint4* __restrict__ k_all, const uint4* __restrict__ v_act,
                                        const int32_t* __restrict__ pos, const int32_t* __restrict__ idx_global,
                                        const int32_t* __restrict__ act_off, int n_seq, int n_act, int row_vec,
                                        BatchCachePtrs c) {
  const size_t total = (size_t)n_act * row_vec;
  for (size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (size_t)gridDim.x * blockDim.x) {
    const int a = (int)(t / row_vec), e = (int)(t - (size_t)a * row_vec);
    int lo = 0, hi = n_seq;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (act_off[mid] <= a) lo = mid; else hi = mid;
    }
    const int i = a - act_off[lo];
    const int src = idx_global[a];
    reinterpret_cast<uint4*>(c.k[lo])[(size_t)i * row_vec + e] = k_all[(size_t)src * row_vec + e];
    reinterpret_cast<uint4*>(c.v[lo])[(size_t)i * row_vec + e] = v_act[(size_t)a * row_vec + e];
    if (e == 0) c.pos[lo][i] = pos[src];
  }
}

// S[n] = (1/H) sum_h exp(l[h, n] - max_h) / sum_h      (Eq. 4)
// `rows` rows of logits contribute; with accumulate the result is added to S (one pass per KV head).
__global__ void pap_mean_kernel(const float* __restrict__ logits, int ld, int N, int rows, int w, int G, float scale,
                                float inv_count, int accumulate, const float* __restrict__ stats,
                                float* __restrict__ S) {
  int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= N) return;
  float acc = 0.f;
  for (int r = 0; r < rows; ++r)
    if (n < pap_row_keys(r, N, w, G)) acc += expf(logits[(size_t)r * ld + n] * scale - stats[2 * r]) / stats[2 * r + 1];
  acc *= inv_count;
  S[n] = accumulate ? S[n] + acc : acc;
}

// q_kv[kvh][i * G + g][:] = q_win[i][(kvh * G + g) * d + :]: the window's queries regrouped by KV head
template <typename T>
__global__ void pap_regroup_kernel(const T* __restrict__ q_win, int w, int Hkv, int G, int d, T* __restrict__ q_kv) {
  const int total = w * Hkv * G * d;
  for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < total; t += gridDim.x * blockDim.x) {
    const int e = t % d, g = (t / d) % G, i = (t / (d * G)) % w, kvh = t / (d * G * w);
    q_kv[t] = q_win[(size_t)i * Hkv * G * d + (size_t)(kvh * G + g) * d + e];
  }
}

__global__ void iota_from_kernel(int32_t* out, int n, int first) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = first + i;
}

// C[n] = sqrt(sum_p csq[n, p]);  S_ffn[n] = C[n] * S_mha[n]      (Eq. 13-14)
__global__ void ffn_score_kernel(const float* __restrict__ csq, int stride, int parts,
                                 const float* __restrict__ S_mha, int N, float* __restrict__ C_out,
                                 float* __restrict__ S_ffn) {
  int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= N) return;
  float s = 0.f;
  for (int p = 0; p < parts; ++p) s += csq[(size_t)n * stride + p];
  float c = sqrtf(fmaxf(s, 0.f));            // the quadratic-form route can round a tiny norm below zero
  if (C_out) C_out[n] = c;
  S_ffn[n] = c * S_mha[n];
}

template <typename T>
__global__ void fold_gain_kernel(T* W, const float* __restrict__ g, size_t total, int in_f) {
  for (size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (size_t)gridDim.x * blockDim.x)
    W[t] = from_f32<T>(to_f32(W[t]) * g[t % in_f]);
}

// out[0] = [vg | 0], out[1] = [0 | vu], each [Dlow, 2r]: lets one dual-weight GEMM evaluate
// silu(t_g Vg) * (t_u Vu) of Eq. 12 from the concatenated low-rank activations [t_g | t_u].
template <typename T>
__global__ void pad_proxy_kernel(const T* __restrict__ vg, const T* __restrict__ vu, int dlow, int r,
                                 T* __restrict__ out) {
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  int total = dlow * 2 * r;
  if (t >= total) return;
  int row = t / (2 * r), c = t - row * 2 * r;
  T zero = from_f32<T>(0.f);
  out[t] = c < r ? vg[row * r + c] : zero;
  out[total + t] = c < r ? zero : vu[row * r + (c - r)];
}

// G = Ud^T Ud for Ud [D, r] (row-major), accumulated in double; written as its bf16 rounding (rows 0..r) followed by
// the bf16 rounding of the remainder (rows r..2r), so that a bf16 tensor-core product with [G_hi ; G_lo] carries G to
// ~2^-17.  One 16 x 16 tile of G per block.  Runs once per layer (spts_prepare_layer) or, without a prepared
// buffer, once per call.
__global__ void gram_kernel(const bf16* __restrict__ ud, int D, int r, bf16* __restrict__ g2) {
  __shared__ float sa[64][17], sb[64][17];
  const int i0 = blockIdx.x * 16, j0 = blockIdx.y * 16;
  const int ti = threadIdx.x & 15, tj = threadIdx.x >> 4;
  double acc = 0.0;
  for (int d0 = 0; d0 < D; d0 += 64) {
    for (int e = threadIdx.x; e < 64 * 16; e += 256) {
      const int dd = e >> 4, c = e & 15;
      const bool in = d0 + dd < D;
      sa[dd][c] = in ? to_f32(ud[(size_t)(d0 + dd) * r + i0 + c]) : 0.f;
      sb[dd][c] = in ? to_f32(ud[(size_t)(d0 + dd) * r + j0 + c]) : 0.f;
    }
    __syncthreads();
    float part = 0.f;                        // 64 products of bf16 pairs: exact enough in fp32 before the double sum
#pragma unroll 16
    for (int dd = 0; dd < 64; ++dd) part = fmaf(sa[dd][ti], sb[dd][tj], part);
    acc += (double)part;
    __syncthreads();
  }
  const float g = (float)acc;
  const bf16 hi = __float2bfloat16_rn(g);
  g2[(size_t)(i0 + ti) * r + j0 + tj] = hi;
  g2[(size_t)(r + i0 + ti) * r + j0 + tj] = __float2bfloat16_rn(g - __bfloat162float(hi));
}

// argmax with the lowest index on ties (NaN never wins; 0 if nothing does), in two steps: every block reduces one
// contiguous share of the logits to (value, index), then one block reduces the shares.
__device__ __forceinline__ void argmax_take(float& best, int& besti, float v, int i) {
  if (v > best || (v == best && i < besti)) { best = v; besti = i; }
}

__device__ __forceinline__ void argmax_block(float& best, int& besti, float* bv, int* bi) {
  const int tid = threadIdx.x;
  for (int o = 16; o > 0; o >>= 1)
    argmax_take(best, besti, __shfl_xor_sync(0xffffffffu, best, o), __shfl_xor_sync(0xffffffffu, besti, o));
  if ((tid & 31) == 0) { bv[tid >> 5] = best; bi[tid >> 5] = besti; }
  __syncthreads();
  if (tid < 32) {
    best = tid < (blockDim.x >> 5) ? bv[tid] : -INFINITY;
    besti = tid < (blockDim.x >> 5) ? bi[tid] : 0x7FFFFFFF;
    for (int o = 16; o > 0; o >>= 1)
      argmax_take(best, besti, __shfl_xor_sync(0xffffffffu, best, o), __shfl_xor_sync(0xffffffffu, besti, o));
  }
}

__global__ void __launch_bounds__(256)
argmax_partial_kernel(const float* __restrict__ logits, int n, float* __restrict__ pv, int* __restrict__ pi) {
  __shared__ float bv[32];
  __shared__ int bi[32];
  const int per = (n + gridDim.x - 1) / gridDim.x;
  const int i0 = blockIdx.x * per, i1 = min(n, i0 + per);
  float best = -INFINITY;
  int besti = 0x7FFFFFFF;
  for (int i = i0 + threadIdx.x; i < i1; i += 4 * 256) {        // four loads in flight per thread
    float v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = i + u * 256 < i1 ? logits[i + u * 256] : -INFINITY;
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (i + u * 256 < i1) argmax_take(best, besti, v[u], i + u * 256);
  }
  argmax_block(best, besti, bv, bi);
  if (threadIdx.x == 0) { pv[blockIdx.x] = best; pi[blockIdx.x] = besti; }
}

__global__ void __launch_bounds__(ARGMAX_BLOCKS)
argmax_final_kernel(const float* __restrict__ pv, const int* __restrict__ pi, int32_t* __restrict__ out) {
  __shared__ float bv[32];
  __shared__ int bi[32];
  float best = pv[threadIdx.x];
  int besti = pi[threadIdx.x];
  if (!(best == best)) { best = -INFINITY; besti = 0x7FFFFFFF; }
  argmax_block(best, besti, bv, bi);
  if (threadIdx.x == 0) *out = besti == 0x7FFFFFFF ? 0 : besti;
}

}  // namespace

spts_status launch_rstd(spts_ctx* ctx, const void* X, int N, float* rstd) {
  const int D = ctx->desc.hidden;
  const int wpb = 8;
  if (ctx->desc.dtype == SPTS_BF16)
    rstd_kernel<bf16><<<ceil_div(N, wpb), wpb * 32, 0, ctx->stream>>>((const bf16*)X, nullptr, N, D, ctx->desc.rms_eps, rstd);
  else
    rstd_kernel<float><<<ceil_div(N, wpb), wpb * 32, 0, ctx->stream>>>((const float*)X, nullptr, N, D, ctx->desc.rms_eps, rstd);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

// rstd[idx[i]] for i < n: the statistic of the listed rows only
spts_status launch_rstd_rows(spts_ctx* ctx, const void* X, const int32_t* idx, int n, float* rstd) {
  const int D = ctx->desc.hidden;
  const int wpb = 8;
  if (n == 0) return SPTS_OK;
  if (ctx->desc.dtype == SPTS_BF16)
    rstd_kernel<bf16><<<ceil_div(n, wpb), wpb * 32, 0, ctx->stream>>>((const bf16*)X, idx, n, D, ctx->desc.rms_eps, rstd);
  else
    rstd_kernel<float><<<ceil_div(n, wpb), wpb * 32, 0, ctx->stream>>>((const float*)X, idx, n, D, ctx->desc.rms_eps, rstd);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_rope_table(spts_ctx* ctx, const int32_t* pos, int N, float2* cs) {
  const int half = ctx->desc.head_dim / 2;
  size_t total = (size_t)N * half;
  rope_table_kernel<<<(unsigned)((total + 255) / 256), 256, 0, ctx->stream>>>(pos, N, half,
                                                                             (double)ctx->desc.rope_theta, cs);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_q_last(spts_ctx* ctx, const void* X, const float2* cs, int N, const void* wq,
                          const float* rstd, float* q) {
  const auto& d = ctx->desc;
  const int HD = d.n_q_heads * d.head_dim;
  const int wpb = 8;
  const int half = d.head_dim / 2;
  dim3 grid(ceil_div(HD / 2, wpb));
  if (d.dtype == SPTS_BF16)
    q_last_kernel<bf16><<<grid, wpb * 32, 0, ctx->stream>>>((const bf16*)X + (size_t)(N - 1) * d.hidden,
        (const bf16*)wq, d.hidden, d.head_dim, HD, 0.f, rstd + (N - 1), cs + (size_t)(N - 1) * half, q, nullptr);
  else
    q_last_kernel<float><<<grid, wpb * 32, 0, ctx->stream>>>((const float*)X + (size_t)(N - 1) * d.hidden,
        (const float*)wq, d.hidden, d.head_dim, HD, 0.f, rstd + (N - 1), cs + (size_t)(N - 1) * half, q, nullptr);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_pap_softmax(spts_ctx* ctx, const float* logits, int ld_logits, int N, float* S) {
  const int H = ctx->desc.n_q_heads;
  pap_head_stats_kernel<<<H, 1024, 0, ctx->stream>>>(logits, ld_logits, N, 1, 1, 1.0f, ctx->ws.head_stats);
  SPTS_CUDA_OK(ctx);
  pap_mean_kernel<<<ceil_div(N, 256), 256, 0, ctx->stream>>>(logits, ld_logits, N, H, 1, 1, 1.0f, 1.0f / (float)H, 0,
                                                            ctx->ws.head_stats, S);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

// One KV head's share of the windowed probe score: logits [w * G, ld] of that head's query rows against all keys
// (raw dot products), softmax per row over its causal range, summed into S with weight 1 / (w * H).
spts_status launch_pap_window_softmax(spts_ctx* ctx, const float* logits, int ld_logits, int N, int w, int accumulate,
                                      float* stats, float* S) {
  const auto& d = ctx->desc;
  const int G = d.n_q_heads / d.n_kv_heads, rows = w * G;
  const float scale = 1.0f / sqrtf((float)d.head_dim);
  pap_head_stats_kernel<<<rows, 1024, 0, ctx->stream>>>(logits, ld_logits, N, w, G, scale, stats);
  SPTS_CUDA_OK(ctx);
  pap_mean_kernel<<<ceil_div(N, 256), 256, 0, ctx->stream>>>(logits, ld_logits, N, rows, w, G, scale,
                                                            1.0f / (float)(w * d.n_q_heads), accumulate, stats, S);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

// out_t[c, r] = in[r, c] for a bf16 matrix [rows, cols] (row stride cols) into [cols, ldt]: the transposed copy of V
// the tensor-core attention reads, for values that did not come out of the library's own V projection.
__global__ void transpose_bf16_kernel(const bf16* __restrict__ in, int rows, int cols, bf16* __restrict__ out_t, int ldt) {
  __shared__ bf16 tile[32][33];
  const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int r = r0 + i, c = c0 + threadIdx.x;
    if (r < rows && c < cols) tile[i][threadIdx.x] = in[(size_t)r * cols + c];
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int c = c0 + i, r = r0 + threadIdx.x;
    if (r < rows && c < cols) out_t[(size_t)c * ldt + r] = tile[threadIdx.x][i];
  }
}

spts_status launch_transpose_bf16(spts_ctx* ctx, const void* in, int rows, int cols, void* out_t, int ldt) {
  if (rows <= 0 || cols <= 0) return SPTS_OK;
  transpose_bf16_kernel<<<dim3(ceil_div(cols, 32), ceil_div(rows, 32)), dim3(32, 8), 0, ctx->stream>>>(
      (const bf16*)in, rows, cols, (bf16*)out_t, ldt);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

// ---- packed batches (tensor-core mode): one launch per step over all sequences
spts_status launch_batch_row_seq(spts_ctx* ctx, const int32_t* seq_start, int n_seq, int total, int32_t* row_seq) {
  batch_row_seq_kernel<<<ceil_div(total, 256), 256, 0, ctx->stream>>>(seq_start, n_seq, total, row_seq);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_batch_vt_col(spts_ctx* ctx, const int32_t* act_off, const int32_t* vt0, int n_seq, int n_act, int32_t* vt_col) {
  if (n_act <= 0) return SPTS_OK;
  batch_vt_col_kernel<<<ceil_div(n_act, 256), 256, 0, ctx->stream>>>(act_off, vt0, n_seq, n_act, vt_col);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_q_last_batch(spts_ctx* ctx, const void* X, const float2* cs, const int32_t* seq_start, int n_seq,
                                const void* wq, const float* rstd, float* q) {
  const auto& d = ctx->desc;
  if (d.dtype != SPTS_BF16) return SPTS_ERR_UNSUPPORTED;
  const int HD = d.n_q_heads * d.head_dim;
  const int wpb = 8;
  dim3 grid(ceil_div(HD / 2, wpb), n_seq);
  q_last_kernel<bf16><<<grid, wpb * 32, 0, ctx->stream>>>((const bf16*)X, (const bf16*)wq, d.hidden, d.head_dim, HD, 0.f,
                                                          rstd, cs, q, seq_start);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_pap_softmax_batch(spts_ctx* ctx, const float* logits, int ld_logits, const int32_t* seq_start,
                                     int n_seq, int total, const int32_t* row_seq, float* stats, float* S) {
  const int H = ctx->desc.n_q_heads;
  pap_head_stats_batch_kernel<<<dim3(H, n_seq), 1024, 0, ctx->stream>>>(logits, ld_logits, seq_start, stats);
  SPTS_CUDA_OK(ctx);
  pap_mean_batch_kernel<<<ceil_div(total, 256), 256, 0, ctx->stream>>>(logits, ld_logits, total, H, row_seq, stats, S);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_batch_cache_fill(spts_ctx* ctx, const void* k_all, const void* v_act, const int32_t* pos,
                                    const int32_t* idx_global, const int32_t* act_off, int n_seq, int n_act,
                                    void* const* k_ptrs, void* const* v_ptrs, int32_t* const* pos_ptrs) {
  const auto& d = ctx->desc;
  const int row_vec = d.n_kv_heads * d.head_dim * 2 / 16;
  if (n_act <= 0) return SPTS_OK;
  size_t total = (size_t)n_act * row_vec;
  int blocks = (int)((total + 255) / 256);
  if (blocks > ctx->sm_count * 16) blocks = ctx->sm_count * 16;
  BatchCachePtrs c{k_ptrs, v_ptrs, pos_ptrs};
  batch_cache_fill_kernel<<<blocks, 256, 0, ctx->stream>>>((const uint4*)k_all, (const uint4*)v_act, pos, idx_global, act_off,
                                                           n_seq, n_act, row_vec, c);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_pap_regroup(spts_ctx* ctx, const void* q_win, int w, void* q_kv) {
  const auto& d = ctx->desc;
  const int G = d.n_q_heads / d.n_kv_heads;
  const int total = w * d.n_q_heads * d.head_dim;
  if (d.dtype == SPTS_BF16)
    pap_regroup_kernel<bf16><<<ceil_div(total, 256), 256, 0, ctx->stream>>>((const bf16*)q_win, w, d.n_kv_heads, G, d.head_dim, (bf16*)q_kv);
  else
    pap_regroup_kernel<float><<<ceil_div(total, 256), 256, 0, ctx->stream>>>((const float*)q_win, w, d.n_kv_heads, G, d.head_dim, (float*)q_kv);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_iota_from(spts_ctx* ctx, int32_t* out, int n, int first) {
  iota_from_kernel<<<ceil_div(n, 256), 256, 0, ctx->stream>>>(out, n, first);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_ffn_score(spts_ctx* ctx, const float* csq, int parts, const float* S_mha, int N,
                             float* C_out, float* S_ffn) {
  ffn_score_kernel<<<ceil_div(N, 256), 256, 0, ctx->stream>>>(csq, ctx->ws.csq_parts, parts, S_mha, N, C_out, S_ffn);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_fold_gain(spts_ctx* ctx, void* W, const float* g, int out_f, int in_f) {
  size_t total = (size_t)out_f * in_f;
  int blocks = (int)((total + 255) / 256);
  if (blocks > ctx->sm_count * 16) blocks = ctx->sm_count * 16;
  if (ctx->desc.dtype == SPTS_BF16)
    fold_gain_kernel<bf16><<<blocks, 256, 0, ctx->stream>>>((bf16*)W, g, total, in_f);
  else
    fold_gain_kernel<float><<<blocks, 256, 0, ctx->stream>>>((float*)W, g, total, in_f);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_pad_proxy(spts_ctx* ctx, const void* vg, const void* vu, void* out) {
  const auto& d = ctx->desc;
  int total = d.ltp_dlow * 2 * d.ltp_rank;
  if (d.dtype == SPTS_BF16)
    pad_proxy_kernel<bf16><<<ceil_div(total, 256), 256, 0, ctx->stream>>>((const bf16*)vg, (const bf16*)vu, d.ltp_dlow, d.ltp_rank, (bf16*)out);
  else
    pad_proxy_kernel<float><<<ceil_div(total, 256), 256, 0, ctx->stream>>>((const float*)vg, (const float*)vu, d.ltp_dlow, d.ltp_rank, (float*)out);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_gram(spts_ctx* ctx, const void* ud, void* g2) {
  const auto& d = ctx->desc;
  if (d.dtype != SPTS_BF16 || d.ltp_rank % 16) return SPTS_ERR_UNSUPPORTED;
  gram_kernel<<<dim3(d.ltp_rank / 16, d.ltp_rank / 16), 256, 0, ctx->stream>>>((const bf16*)ud, d.hidden, d.ltp_rank, (bf16*)g2);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_head(spts_ctx* ctx, const void* x_row, const void* lm_head, float* logits,
                        int32_t* token_out) {
  // the row is widened into the fp32 vector scratch that the decode kernels use, then the same
  // weight-streaming matrix-vector kernel computes rstd(x) * lm_head x
  spts_status s = launch_decode_load(ctx, x_row);
  if (s != SPTS_OK) return s;
  s = launch_head_logits(ctx, (const float*)ctx->ws.dec, lm_head, logits);
  if (s != SPTS_OK) return s;
  if (token_out != nullptr) {
    float* pv = argmax_scratch(ctx);
    int* pi = (int*)(pv + ARGMAX_BLOCKS);
    argmax_partial_kernel<<<ARGMAX_BLOCKS, 256, 0, ctx->stream>>>(logits, ctx->desc.vocab, pv, pi);
    SPTS_CUDA_OK(ctx);
    argmax_final_kernel<<<1, ARGMAX_BLOCKS, 0, ctx->stream>>>(pv, pi, token_out);
    SPTS_CUDA_OK(ctx);
  }
  return SPTS_OK;
}

}  // namespace spts
