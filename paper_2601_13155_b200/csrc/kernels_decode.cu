// Decode step (Algorithm 1 outside the prefill phase): one new token runs every layer densely
// against that layer's compressed KV cache plus itself.  Batch-1 decode streams every weight
// once, so all kernels here are HBM-bound matrix-vector products with 16-byte loads; the
// residual vector lives in fp32 scratch and is rounded through the storage type at the same
// points as the prefill path.
#include "spts_common.cuh"

namespace spts {

namespace {

template <typename T> struct DV;
template <> struct DV<float> { static constexpr int N = 4; };
template <> struct DV<bf16> { static constexpr int N = 8; };

template <typename T> __device__ __forceinline__ void ld16(const T* p, float* out);
template <> __device__ __forceinline__ void ld16<float>(const float* p, float* out) {
  float4 v = *reinterpret_cast<const float4*>(p);
  out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
template <> __device__ __forceinline__ void ld16<bf16>(const bf16* p, float* out) {
  uint4 v = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out[2 * i] = __uint_as_float(w[i] << 16);
    out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

template <typename T> __device__ __forceinline__ float round_through(float v) { return to_f32(from_f32<T>(v)); }

template <typename T>
__global__ void vec_load_kernel(const T* __restrict__ x, int D, float* __restrict__ out) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < D) out[i] = to_f32(x[i]);
}
template <typename T>
__global__ void vec_store_kernel(const float* __restrict__ x, int D, T* __restrict__ out) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < D) out[i] = from_f32<T>(x[i]);
}

// out[j] (op)= scale * sum_k xin[k] W[j, k], with scale = rstd(xin) when NORM.
// RESID: out[j] = round(out[j] + dot).  One warp per output row; xin staged in shared memory.
template <typename T, bool NORM, bool RESID>
__global__ void __launch_bounds__(256)
gemv_kernel(const T* __restrict__ W, int rows, int K, const float* __restrict__ xin, float eps,
            float* __restrict__ out) {
  constexpr int V = DV<T>::N;
  extern __shared__ float xs[];
  __shared__ float red[8];
  __shared__ float rs_sh;
  const int tid = threadIdx.x;
  float ss = 0.f;
  for (int c = tid; c < K; c += blockDim.x) { float v = xin[c]; xs[c] = v; ss = fmaf(v, v, ss); }
  if (NORM) {
    ss = warp_sum(ss);
    if ((tid & 31) == 0) red[tid >> 5] = ss;
    __syncthreads();
    if (tid == 0) {
      float v = 0.f;
      for (int w = 0; w < 8; ++w) v += red[w];
      rs_sh = 1.0f / sqrtf(v / (float)K + eps);
    }
  }
  __syncthreads();
  const int row = blockIdx.x * 8 + (tid >> 5);
  if (row >= rows) return;
  const int lane = tid & 31;
  const T* w = W + (size_t)row * K;
  float a = 0.f;
  for (int c = lane * V; c < K; c += 32 * V) {
    float u[V];
    ld16<T>(w + c, u);
#pragma unroll
    for (int e = 0; e < V; ++e) a = fmaf(xs[c + e], u[e], a);
  }
  a = warp_sum(a);
  if (lane == 0) {
    if (NORM) a *= rs_sh;
    if (RESID) out[row] = round_through<T>(out[row] + a);
    else out[row] = a;
  }
}

// RoPE on q and k of the new token, rounding through the storage type; append k, v, pos to the cache.
template <typename T>
__global__ void dec_rope_store_kernel(float* __restrict__ q32, const float* __restrict__ k32,
                                      const float* __restrict__ v32, int H, int Hkv, int d, int pos,
                                      double theta, T* __restrict__ kc, T* __restrict__ vc,
                                      int32_t* __restrict__ pc, int slot) {
  int half = d >> 1;
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  int nq = H * half, nk = Hkv * half;
  if (t < nq + nk) {
    bool isq = t < nq;
    int u = isq ? t : t - nq;
    int h = u / half, i = u - h * half;
    double inv = exp2(-(double)(2 * i) / (double)d * log2(theta));
    double s, c;
    sincos((double)pos * inv, &s, &c);
    float cf = (float)c, sf = (float)s;
    const float* src = isq ? q32 : k32;
    float a = src[h * d + i], b = src[h * d + i + half];
    float r1 = a * cf - b * sf, r2 = b * cf + a * sf;
    if (isq) {
      q32[h * d + i] = round_through<T>(r1);
      q32[h * d + i + half] = round_through<T>(r2);
    } else {
      kc[((size_t)slot * Hkv + h) * d + i] = from_f32<T>(r1);
      kc[((size_t)slot * Hkv + h) * d + i + half] = from_f32<T>(r2);
    }
  }
  if (t < Hkv * d) vc[(size_t)slot * Hkv * d + t] = from_f32<T>(v32[t]);
  if (t == 0) pc[slot] = pos;
}

// Split-KV attention of one query: block (h, s) handles keys [s*len/ns, (s+1)*len/ns).
// part[(h*ns + s)] = (max, sum, o[d]); 4 warps, each strides over keys; lane owns d/32 dims.
template <typename T, int DPL>
__global__ void __launch_bounds__(128)
dec_attn_partial_kernel(const float* __restrict__ q32, const T* __restrict__ kc, const T* __restrict__ vc,
                        int len, int H, int Hkv, int nsplit, float* __restrict__ part) {
  constexpr int d = DPL * 32;
  __shared__ float sm_m[4], sm_l[4], sm_o[4][d];
  const int h = blockIdx.x, s = blockIdx.y;
  const int kvh = h / (H / Hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j0 = (int)((long)len * s / nsplit), j1 = (int)((long)len * (s + 1) / nsplit);
  const float scale = rsqrtf((float)d);
  float qv[DPL];
#pragma unroll
  for (int c = 0; c < DPL; ++c) qv[c] = q32[h * d + c * 32 + lane] * scale;
  float m = -INFINITY, l = 0.f, o[DPL];
#pragma unroll
  for (int c = 0; c < DPL; ++c) o[c] = 0.f;
  for (int j = j0 + warp; j < j1; j += 4) {
    const T* kr = kc + ((size_t)j * Hkv + kvh) * d;
    const T* vr = vc + ((size_t)j * Hkv + kvh) * d;
    float dot = 0.f;
#pragma unroll
    for (int c = 0; c < DPL; ++c) dot = fmaf(qv[c], to_f32(kr[c * 32 + lane]), dot);
    dot = warp_sum(dot);
    float mn = fmaxf(m, dot);
    float corr = expf(m - mn), p = expf(dot - mn);
    l = l * corr + p;
#pragma unroll
    for (int c = 0; c < DPL; ++c) o[c] = fmaf(p, to_f32(vr[c * 32 + lane]), o[c] * corr);
    m = mn;
  }
  if (lane == 0) { sm_m[warp] = m; sm_l[warp] = l; }
#pragma unroll
  for (int c = 0; c < DPL; ++c) sm_o[warp][c * 32 + lane] = o[c];
  __syncthreads();
  if (warp == 0) {
    float M = fmaxf(fmaxf(sm_m[0], sm_m[1]), fmaxf(sm_m[2], sm_m[3]));
    float L = 0.f, acc[DPL];
#pragma unroll
    for (int c = 0; c < DPL; ++c) acc[c] = 0.f;
    for (int w = 0; w < 4; ++w) {
      float f = sm_m[w] == -INFINITY ? 0.f : expf(sm_m[w] - M);
      L += sm_l[w] * f;
#pragma unroll
      for (int c = 0; c < DPL; ++c) acc[c] = fmaf(sm_o[w][c * 32 + lane], f, acc[c]);
    }
    float* p = part + ((size_t)h * nsplit + s) * (d + 2);
    if (lane == 0) { p[0] = M; p[1] = L; }
#pragma unroll
    for (int c = 0; c < DPL; ++c) p[2 + c * 32 + lane] = acc[c];
  }
}

template <typename T>
__global__ void dec_attn_combine_kernel(const float* __restrict__ part, int nsplit, int d,
                                        float* __restrict__ att32) {
  const int h = blockIdx.x, t = threadIdx.x;   // blockDim = d
  float M = -INFINITY;
  for (int s = 0; s < nsplit; ++s) M = fmaxf(M, part[((size_t)h * nsplit + s) * (d + 2)]);
  float L = 0.f, acc = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    const float* p = part + ((size_t)h * nsplit + s) * (d + 2);
    float f = p[0] == -INFINITY ? 0.f : expf(p[0] - M);
    L += p[1] * f;
    acc = fmaf(p[2 + t], f, acc);
  }
  att32[h * d + t] = round_through<T>(acc / L);
}

template <typename T>
__global__ void dec_swiglu_kernel(const float* __restrict__ g, const float* __restrict__ u, int n,
                                  float* __restrict__ out) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    float a = g[i];
    out[i] = round_through<T>(a / (1.0f + expf(-a)) * u[i]);
  }
}

constexpr int DEC_MAX_SPLIT = 64;

template <typename T>
spts_status decode_layer_t(spts_ctx* ctx, const spts_layer_weights* w, spts_kv_layer* cache, float* x32,
                           int32_t pos) {
  const auto& d = ctx->desc;
  cudaStream_t st = ctx->stream;
  const int D = d.hidden, H = d.n_q_heads, Hkv = d.n_kv_heads, hd = d.head_dim, Dff = d.ffn_dim;
  float* base = (float*)ctx->ws.dec;
  float* q32 = base + D;                     // [H*hd]
  float* k32 = q32 + H * hd;                 // [Hkv*hd]
  float* v32 = k32 + Hkv * hd;               // [Hkv*hd]
  float* att32 = v32 + Hkv * hd;             // [H*hd]
  float* g32 = att32 + H * hd;               // [Dff]
  float* u32 = g32 + Dff;                    // [Dff]
  float* hm32 = u32 + Dff;                   // [Dff]
  float* part = hm32 + Dff;                  // [H, DEC_MAX_SPLIT, hd + 2]
  if (cache->len + 1 > cache->capacity) return SPTS_ERR_WORKSPACE;
  const size_t smD = (size_t)D * 4;
  gemv_kernel<T, true, false><<<ceil_div(H * hd, 8), 256, smD, st>>>((const T*)w->wq, H * hd, D, x32, d.rms_eps, q32);
  SPTS_CUDA_OK(ctx);
  gemv_kernel<T, true, false><<<ceil_div(Hkv * hd, 8), 256, smD, st>>>((const T*)w->wk, Hkv * hd, D, x32, d.rms_eps, k32);
  SPTS_CUDA_OK(ctx);
  gemv_kernel<T, true, false><<<ceil_div(Hkv * hd, 8), 256, smD, st>>>((const T*)w->wv, Hkv * hd, D, x32, d.rms_eps, v32);
  SPTS_CUDA_OK(ctx);
  const int slot = cache->len;
  int nthr = max(H * hd / 2 + Hkv * hd / 2, Hkv * hd);
  dec_rope_store_kernel<T><<<ceil_div(nthr, 256), 256, 0, st>>>(q32, k32, v32, H, Hkv, hd, pos, (double)d.rope_theta,
                                                              (T*)cache->k, (T*)cache->v, cache->pos, slot);
  SPTS_CUDA_OK(ctx);
  cache->len = slot + 1;
  const int len = cache->len;
  int nsplit = min(DEC_MAX_SPLIT, max(1, len / 256));
  dim3 grid(H, nsplit);
  if (hd == 128) dec_attn_partial_kernel<T, 4><<<grid, 128, 0, st>>>(q32, (const T*)cache->k, (const T*)cache->v, len, H, Hkv, nsplit, part);
  else dec_attn_partial_kernel<T, 2><<<grid, 128, 0, st>>>(q32, (const T*)cache->k, (const T*)cache->v, len, H, Hkv, nsplit, part);
  SPTS_CUDA_OK(ctx);
  dec_attn_combine_kernel<T><<<H, hd, 0, st>>>(part, nsplit, hd, att32);
  SPTS_CUDA_OK(ctx);
  gemv_kernel<T, false, true><<<ceil_div(D, 8), 256, (size_t)H * hd * 4, st>>>((const T*)w->wo, D, H * hd, att32, 0.f, x32);
  SPTS_CUDA_OK(ctx);
  gemv_kernel<T, true, false><<<ceil_div(Dff, 8), 256, smD, st>>>((const T*)w->w_gate, Dff, D, x32, d.rms_eps, g32);
  SPTS_CUDA_OK(ctx);
  gemv_kernel<T, true, false><<<ceil_div(Dff, 8), 256, smD, st>>>((const T*)w->w_up, Dff, D, x32, d.rms_eps, u32);
  SPTS_CUDA_OK(ctx);
  dec_swiglu_kernel<T><<<ceil_div(Dff, 256), 256, 0, st>>>(g32, u32, Dff, hm32);
  SPTS_CUDA_OK(ctx);
  if ((size_t)Dff * 4 > 48 * 1024) {
    cudaFuncSetAttribute(gemv_kernel<T, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Dff * 4);
  }
  gemv_kernel<T, false, true><<<ceil_div(D, 8), 256, (size_t)Dff * 4, st>>>((const T*)w->w_down, D, Dff, hm32, 0.f, x32);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

}  // namespace

size_t decode_scratch_floats(const spts_model_desc& d) {
  return (size_t)d.hidden + 2 * (size_t)d.n_q_heads * d.head_dim + 2 * (size_t)d.n_kv_heads * d.head_dim +
         3 * (size_t)d.ffn_dim + (size_t)d.n_q_heads * DEC_MAX_SPLIT * (d.head_dim + 2) + 64;
}

spts_status launch_decode_load(spts_ctx* ctx, const void* x) {
  const int D = ctx->desc.hidden;
  float* x32 = (float*)ctx->ws.dec;
  if (ctx->desc.dtype == SPTS_BF16) vec_load_kernel<bf16><<<ceil_div(D, 256), 256, 0, ctx->stream>>>((const bf16*)x, D, x32);
  else vec_load_kernel<float><<<ceil_div(D, 256), 256, 0, ctx->stream>>>((const float*)x, D, x32);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_decode_store(spts_ctx* ctx, void* x) {
  const int D = ctx->desc.hidden;
  float* x32 = (float*)ctx->ws.dec;
  if (ctx->desc.dtype == SPTS_BF16) vec_store_kernel<bf16><<<ceil_div(D, 256), 256, 0, ctx->stream>>>(x32, D, (bf16*)x);
  else vec_store_kernel<float><<<ceil_div(D, 256), 256, 0, ctx->stream>>>(x32, D, (float*)x);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_decode_layer(spts_ctx* ctx, const spts_layer_weights* w, spts_kv_layer* cache, int32_t pos) {
  float* x32 = (float*)ctx->ws.dec;
  if (ctx->desc.dtype == SPTS_BF16) return decode_layer_t<bf16>(ctx, w, cache, x32, pos);
  return decode_layer_t<float>(ctx, w, cache, x32, pos);
}

}  // namespace spts
