// Plain CUDA-core kernels: the fp32 verification mode of the library, and an on-GPU cross-check
// for the tensor-core path in bf16 mode.  Storage type T (float or bf16), fp32 arithmetic, the
// same rounding points as the tensor-core kernels.
//
//   ref_gemm:      acc[i, j] = sum_k A[src(i), k] * W[j, k]   with fused epilogues
//   ref_attention: causal GQA attention among m rows (Algorithm 1, reduced MHA)
#include "spts_common.cuh"

namespace spts {

namespace {

constexpr int RB = 64;    // tile rows / cols
constexpr int RK = 16;    // k-step
constexpr int RT = 256;   // threads (16 x 16), 4 x 4 outputs each

template <typename T, int EPI>
__global__ void __launch_bounds__(RT)
ref_gemm_kernel(RefGemmArgs a, const float2* __restrict__ cs, float* __restrict__ aux32) {
  constexpr bool DUAL = (EPI == REF_ROPE || EPI == REF_SWIGLU);
  __shared__ float As[RK][RB + 4];
  __shared__ float Bs[RK][RB + 4];
  __shared__ float B2s[DUAL ? RK : 1][RB + 4];
  __shared__ float red[RB][17];
  const T* A = (const T*)a.A;
  const T* W = (const T*)a.W;
  const T* W2 = (const T*)a.W2;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int row0 = blockIdx.y * RB, col0 = blockIdx.x * RB;
  const int half = a.head_dim >> 1;
  const long ldw = a.ldw ? a.ldw : a.K;

  // loader mapping: thread -> (tile row r, 4 consecutive k)
  const int lr = tid >> 2, lk = (tid & 3) * 4;
  const int gi = row0 + lr;
  long a_row = -1;
  if (gi < a.M) a_row = a.idx ? (long)a.idx[gi] : (long)gi;
  const int gj = col0 + lr;
  long w_row = gj < a.Nout ? (long)gj : -1;
  long w2_row = -1;
  if (DUAL && gj < a.Nout) {
    if (EPI == REF_ROPE) {
      int jj = gj % a.head_dim;
      w2_row = jj < half ? gj + half : gj - half;   // rotary partner column
    } else {
      w2_row = gj;
    }
  }
  const T* Wsec = (EPI == REF_ROPE) ? W : W2;

  float acc[4][4], acc2[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { acc[i][j] = 0.f; acc2[i][j] = 0.f; }

  for (int k0 = 0; k0 < a.K; k0 += RK) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      int k = k0 + lk + e;
      float va = 0.f, vb = 0.f, vb2 = 0.f;
      if (k < a.K) {
        if (a_row >= 0) va = to_f32(A[a_row * a.lda + k]);
        if (w_row >= 0) vb = to_f32(W[w_row * ldw + k]);
        if (DUAL && w2_row >= 0) vb2 = to_f32(Wsec[w2_row * ldw + k]);
      }
      As[lk + e][lr] = va;
      Bs[lk + e][lr] = vb;
      if (DUAL) B2s[lk + e][lr] = vb2;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < RK; ++k) {
      float av[4], bv[4], b2v[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) { bv[j] = Bs[k][tx * 4 + j]; if (DUAL) b2v[j] = B2s[k][tx * 4 + j]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
          if (DUAL) acc2[i][j] = fmaf(av[i], b2v[j], acc2[i][j]);
        }
    }
    __syncthreads();
  }

  // ---- epilogue
  T* out = (T*)a.out;
  if (EPI == REF_SUMSQ) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float s = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int gj2 = col0 + tx * 4 + j;
        if (gj2 < a.Nout) s = fmaf(acc[i][j], acc[i][j], s);
      }
      red[ty * 4 + i][tx] = s;
    }
    __syncthreads();
    if (tid < RB) {
      int gi2 = row0 + tid;
      if (gi2 < a.M) {
        float s = 0.f;
        for (int t = 0; t < 16; ++t) s += red[tid][t];
        a.csq[(size_t)gi2 * a.csq_parts + blockIdx.x] = s;
      }
    }
    return;
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int gi2 = row0 + ty * 4 + i;
    if (gi2 >= a.M) continue;
    long src = a.idx ? (long)a.idx[gi2] : (long)gi2;
    float rs = a.rowscale ? a.rowscale[src] : 1.0f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int gj2 = col0 + tx * 4 + j;
      if (gj2 >= a.Nout) continue;
      float v = acc[i][j] * rs;
      if (EPI == REF_STORE) {
        if (a.out_f32 != nullptr) { a.out_f32[(size_t)gi2 * a.ldo + gj2] = v; continue; }
        T o = from_f32<T>(v);
        out[(size_t)gi2 * a.ldo + gj2] = o;
        if (a.out_t) ((T*)a.out_t)[(size_t)gj2 * a.ldt + gi2] = o;
      } else if (EPI == REF_ROPE) {
        float v2 = acc2[i][j] * rs;
        int jj = gj2 % a.head_dim;
        float2 c = cs[(size_t)src * half + (jj % half)];
        float r = jj < half ? v * c.x - v2 * c.y : v * c.x + v2 * c.y;
        out[(size_t)gi2 * a.ldo + gj2] = from_f32<T>(r);
        if (aux32) aux32[(size_t)gi2 * a.Nout + gj2] = r;   // unrounded keys for the PAP logits
      } else if (EPI == REF_SWIGLU) {
        float u = acc2[i][j] * rs;
        float g = v / (1.0f + expf(-v));
        if (a.sal_t != nullptr) a.sal_t[(size_t)gj2 * a.ld_sal + gi2] = fabsf(g * u);
        else out[(size_t)gi2 * a.ldo + gj2] = from_f32<T>(g * u);
      } else if (EPI == REF_RESID) {
        long dst = a.dst_idx ? (long)a.dst_idx[gi2] : (long)gi2;
        size_t o = (size_t)dst * a.ldo + gj2;
        out[o] = from_f32<T>(to_f32(out[o]) + acc[i][j]);
      }
    }
  }
}

// logits[h, n] = q[h] . K32[n, h / group] / sqrt(d); one warp per (n, h)
__global__ void ref_pap_logits_kernel(const float* __restrict__ K32, const float* __restrict__ q, int N,
                                      int H, int Hkv, int d, float* __restrict__ logits, int ld) {
  int w = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (w >= N * H) return;
  int n = w / H, h = w - n * H;
  int lane = threadIdx.x & 31;
  const float* k = K32 + ((size_t)n * Hkv + h / (H / Hkv)) * d;
  const float* qq = q + (size_t)h * d;
  float s = 0.f;
  for (int t = lane; t < d; t += 32) s = fmaf(qq[t], k[t], s);
  s = warp_sum(s);
  if (lane == 0) logits[(size_t)h * ld + n] = s * rsqrtf((float)d);
}

// One warp per (query row i, head h): online-softmax attention over keys j <= i.
template <typename T, int DPL>   // DPL = head_dim / 32 output dims per lane
__global__ void __launch_bounds__(128)
ref_attention_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V, int m,
                     int H, int Hkv, T* __restrict__ O) {
  constexpr int d = DPL * 32;
  __shared__ float qs[4][d];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = blockIdx.x;
  const int h = blockIdx.y * 4 + warp;
  if (h >= H) return;
  const int kvh = h / (H / Hkv);
  const float scale = rsqrtf((float)d);
  for (int t = lane; t < d; t += 32) qs[warp][t] = to_f32(Q[((size_t)i * H + h) * d + t]) * scale;
  __syncwarp();
  float mrun = -INFINITY, lrun = 0.f;
  float o[DPL];
#pragma unroll
  for (int c = 0; c < DPL; ++c) o[c] = 0.f;
  for (int j0 = 0; j0 <= i; j0 += 32) {
    int j = j0 + lane;
    float s = -INFINITY;
    if (j <= i) {
      const T* kr = K + ((size_t)j * Hkv + kvh) * d;
      float acc = 0.f;
      for (int t = 0; t < d; ++t) acc = fmaf(qs[warp][t], to_f32(kr[t]), acc);
      s = acc;
    }
    float mnew = fmaxf(mrun, warp_max(s));
    float p = j <= i ? expf(s - mnew) : 0.f;
    float corr = expf(mrun - mnew);
    lrun = lrun * corr + warp_sum(p);
    mrun = mnew;
#pragma unroll
    for (int c = 0; c < DPL; ++c) o[c] *= corr;
    int cnt = min(32, i - j0 + 1);
    for (int l = 0; l < cnt; ++l) {
      float pj = __shfl_sync(0xffffffffu, p, l);
      const T* vr = V + ((size_t)(j0 + l) * Hkv + kvh) * d;
#pragma unroll
      for (int c = 0; c < DPL; ++c) o[c] = fmaf(pj, to_f32(vr[c * 32 + lane]), o[c]);
    }
  }
  float inv = 1.0f / lrun;
#pragma unroll
  for (int c = 0; c < DPL; ++c) O[((size_t)i * H + h) * d + c * 32 + lane] = from_f32<T>(o[c] * inv);
}

template <typename T>
spts_status ref_gemm_dispatch(spts_ctx* ctx, int epi, const RefGemmArgs& a, const float2* cs, float* aux32) {
  dim3 grid(ceil_div(a.Nout, RB), ceil_div(a.M, RB));
  cudaStream_t st = ctx->stream;
  switch (epi) {
    case REF_STORE: ref_gemm_kernel<T, REF_STORE><<<grid, RT, 0, st>>>(a, cs, aux32); break;
    case REF_ROPE: ref_gemm_kernel<T, REF_ROPE><<<grid, RT, 0, st>>>(a, cs, aux32); break;
    case REF_SWIGLU: ref_gemm_kernel<T, REF_SWIGLU><<<grid, RT, 0, st>>>(a, cs, aux32); break;
    case REF_RESID: ref_gemm_kernel<T, REF_RESID><<<grid, RT, 0, st>>>(a, cs, aux32); break;
    case REF_SUMSQ: ref_gemm_kernel<T, REF_SUMSQ><<<grid, RT, 0, st>>>(a, cs, aux32); break;
    default: return SPTS_ERR_INVALID_ARG;
  }
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

}  // namespace

spts_status launch_ref_gemm(spts_ctx* ctx, int epi, const RefGemmArgs& a) {
  if (a.M <= 0) return SPTS_OK;
  if (epi == REF_SUMSQ && ceil_div(a.Nout, RB) > a.csq_parts) return SPTS_ERR_WORKSPACE;
  const bool pap = (epi == REF_ROPE && a.logits != nullptr);
  float* aux = nullptr;
  if (pap) {
    if ((size_t)a.M * a.Nout > ctx->ws.acc32_elems) return SPTS_ERR_WORKSPACE;
    aux = ctx->ws.acc32;
  }
  spts_status s = ctx->desc.dtype == SPTS_BF16 ? ref_gemm_dispatch<bf16>(ctx, epi, a, ctx->ws.rope_cs, aux)
                                               : ref_gemm_dispatch<float>(ctx, epi, a, ctx->ws.rope_cs, aux);
  if (s != SPTS_OK) return s;
  if (pap) {
    const auto& d = ctx->desc;
    int warps = a.M * d.n_q_heads;
    ref_pap_logits_kernel<<<ceil_div(warps, 8), 256, 0, ctx->stream>>>(aux, a.q, a.M, d.n_q_heads, d.n_kv_heads,
                                                                       d.head_dim, a.logits, a.ld_logits);
    SPTS_CUDA_OK(ctx);
  }
  return SPTS_OK;
}

spts_status launch_ref_attention(spts_ctx* ctx, const void* Q, const void* K, const void* V, int m, void* O) {
  if (m <= 0) return SPTS_OK;
  const auto& d = ctx->desc;
  dim3 grid(m, ceil_div(d.n_q_heads, 4));
  cudaStream_t st = ctx->stream;
  if (d.dtype == SPTS_BF16) {
    if (d.head_dim == 128)
      ref_attention_kernel<bf16, 4><<<grid, 128, 0, st>>>((const bf16*)Q, (const bf16*)K, (const bf16*)V, m, d.n_q_heads, d.n_kv_heads, (bf16*)O);
    else
      ref_attention_kernel<bf16, 2><<<grid, 128, 0, st>>>((const bf16*)Q, (const bf16*)K, (const bf16*)V, m, d.n_q_heads, d.n_kv_heads, (bf16*)O);
  } else {
    if (d.head_dim == 128)
      ref_attention_kernel<float, 4><<<grid, 128, 0, st>>>((const float*)Q, (const float*)K, (const float*)V, m, d.n_q_heads, d.n_kv_heads, (float*)O);
    else
      ref_attention_kernel<float, 2><<<grid, 128, 0, st>>>((const float*)Q, (const float*)K, (const float*)V, m, d.n_q_heads, d.n_kv_heads, (float*)O);
  }
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

}  // namespace spts
