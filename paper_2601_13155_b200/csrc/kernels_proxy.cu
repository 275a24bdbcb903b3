// Offline construction of the low-rank proxy FFN (Section 3.3 of the SPTS paper): channel importance
// from the calibration saliencies, the reduced projection matrices W' = W[:, C], and their rank-r
// factorisation W' ~ U V by a one-sided Jacobi SVD.  fp32 arithmetic; runs once per layer, off the
// inference path, but on the GPU and behind the same C boundary.
#include "spts_common.cuh"

namespace spts {

namespace {

// ---------------------------------------------------------------------------------------------
// I_j = mean of the k largest saliency values of channel j over the calibration tokens.
// One CTA per channel; zt [Dff, ld] holds one row of n non-negative values per channel.  The k-th
// largest value T is found by an 8-bit radix select on the float bit patterns (monotone for
// non-negative floats); I_j = (sum of values > T + (k - #{> T}) * T) / k.
// ---------------------------------------------------------------------------------------------
constexpr int IMP_THREADS = 256;

__global__ void __launch_bounds__(IMP_THREADS)
proxy_importance_kernel(const float* __restrict__ zt, int ld, int n, int k, float* __restrict__ importance) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t sel_prefix, sel_krem;
  __shared__ float red[IMP_THREADS / 32];
  __shared__ uint32_t redc[IMP_THREADS / 32];
  const float* z = zt + (size_t)blockIdx.x * ld;
  const int tid = threadIdx.x;
  uint32_t prefix = 0, krem = (uint32_t)k;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const uint32_t mask = pass == 0 ? 0u : (0xFFFFFFFFu << (32 - 8 * pass));
    hist[tid] = 0;
    __syncthreads();
    for (int i = tid; i < n; i += IMP_THREADS) {
      const uint32_t key = __float_as_uint(z[i]) & 0x7FFFFFFFu;
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 0xFFu], 1u);
    }
    __syncthreads();
    if (tid == 0) {          // walk the buckets from the top: 256 steps, once per pass
      uint32_t above = 0;
      int b = 255;
      for (; b > 0; --b) {
        if (above + hist[b] >= krem) break;
        above += hist[b];
      }
      sel_prefix = prefix | ((uint32_t)b << shift);
      sel_krem = krem - above;
    }
    __syncthreads();
    prefix = sel_prefix;
    krem = sel_krem;
    __syncthreads();
  }
  const float T = __uint_as_float(prefix);
  float s = 0.f;
  uint32_t cnt = 0;
  for (int i = tid; i < n; i += IMP_THREADS) {
    const float v = fabsf(z[i]);
    if (v > T) { s += v; ++cnt; }
  }
  s = warp_sum(s);
  cnt = __reduce_add_sync(0xffffffffu, cnt);
  if ((tid & 31) == 0) { red[tid >> 5] = s; redc[tid >> 5] = cnt; }
  __syncthreads();
  if (tid == 0) {
    float S = 0.f;
    uint32_t Cn = 0;
    for (int w = 0; w < IMP_THREADS / 32; ++w) { S += red[w]; Cn += redc[w]; }
    importance[blockIdx.x] = (S + (float)((uint32_t)k - Cn) * T) / (float)k;
  }
}

// ---------------------------------------------------------------------------------------------
// Reduced matrices in fp32, one column of W' (length D) per row of the work array:
//   gate / up:  A[c, :] = W[C[c], :]          (W stored [Dff, D])
//   down:       A[c, d] = W[d, C[c]]          (W stored [D, Dff])
// and V starts as the identity [n, n].
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void proxy_slice_kernel(const T* __restrict__ W, const int32_t* __restrict__ C, int n, int D, int Dff,
                                   int down, float* __restrict__ A, float* __restrict__ V) {
  const int c = blockIdx.x;
  const int ch = C[c];
  for (int d = threadIdx.x; d < D; d += blockDim.x)
    A[(size_t)c * D + d] = down ? to_f32(W[(size_t)d * Dff + ch]) : to_f32(W[(size_t)ch * D + d]);
  for (int j = threadIdx.x; j < n; j += blockDim.x) V[(size_t)c * n + j] = j == c ? 1.0f : 0.0f;
}

// ---------------------------------------------------------------------------------------------
// One-sided (Hestenes) Jacobi SVD.  The n columns of W' are the rows a_c of A [n, m]; a rotation of
// the pair (p, q) makes a_p and a_q orthogonal and is applied to the rows of V [n, n] as well, so at
// the end A = G A_0 with orthogonal rows (a_c = sigma_c u_c) and V = G:  W' = sum_c u_c sigma_c V[c, :].
// One launch = one round of the round-robin ordering: n / 2 disjoint pairs, one CTA each.
// ---------------------------------------------------------------------------------------------
constexpr int JAC_THREADS = 256;

__device__ __forceinline__ double block_sum(double v, double* red) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();                                     // red[] may still be read from the previous call
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  double s = 0.0;
#pragma unroll
  for (int w = 0; w < JAC_THREADS / 32; ++w) s += red[w];
  return s;
}

__global__ void __launch_bounds__(JAC_THREADS)
proxy_jacobi_round_kernel(float* __restrict__ A, float* __restrict__ V, int n, int m, int round,
                          unsigned int* __restrict__ offdiag) {
  __shared__ double red[JAC_THREADS / 32];
  const int i = blockIdx.x;                            // slot of the round: circle method on n - 1 players + 1 fixed
  int p, q;
  if (i == 0) { p = n - 1; q = round % (n - 1); }
  else { p = (round + i) % (n - 1); q = (round - i + (n - 1)) % (n - 1); }
  if (p > q) { const int t = p; p = q; q = t; }
  float* ap = A + (size_t)p * m;
  float* aq = A + (size_t)q * m;
  float a = 0.f, b = 0.f, g = 0.f;
  for (int d = threadIdx.x; d < m; d += JAC_THREADS) {
    const float x = ap[d], y = aq[d];
    a = fmaf(x, x, a); b = fmaf(y, y, b); g = fmaf(x, y, g);
  }
  const double alpha = block_sum((double)a, red), beta = block_sum((double)b, red), gamma = block_sum((double)g, red);
  const double denom = sqrt(alpha * beta);
  if (!(denom > 0.0)) return;                          // a zero column: nothing to rotate
  const double rel = fabs(gamma) / denom;
  if (threadIdx.x == 0) atomicMax(offdiag, __float_as_uint((float)rel));
  if (rel <= 1e-9) return;
  const double zeta = (beta - alpha) / (2.0 * gamma);
  const double t = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
  const double cd = 1.0 / sqrt(1.0 + t * t);
  const float c = (float)cd, s = (float)(cd * t);
  for (int d = threadIdx.x; d < m; d += JAC_THREADS) {
    const float x = ap[d], y = aq[d];
    ap[d] = c * x - s * y;
    aq[d] = s * x + c * y;
  }
  float* vp = V + (size_t)p * n;
  float* vq = V + (size_t)q * n;
  for (int d = threadIdx.x; d < n; d += JAC_THREADS) {
    const float x = vp[d], y = vq[d];
    vp[d] = c * x - s * y;
    vq[d] = s * x + c * y;
  }
}

// sigma[c] = || a_c ||
__global__ void __launch_bounds__(JAC_THREADS)
proxy_sigma_kernel(const float* __restrict__ A, int m, float* __restrict__ sigma) {
  __shared__ double red[JAC_THREADS / 32];
  const float* a = A + (size_t)blockIdx.x * m;
  float s = 0.f;
  for (int d = threadIdx.x; d < m; d += JAC_THREADS) s = fmaf(a[d], a[d], s);
  const double tot = block_sum((double)s, red);
  if (threadIdx.x == 0) sigma[blockIdx.x] = (float)sqrt(tot);
}

// order[k] = index of the k-th largest sigma (ties to the lower index); sigma_sorted[k] its value
__global__ void proxy_rank_kernel(const float* __restrict__ sigma, int n, int32_t* __restrict__ order,
                                  float* __restrict__ sigma_sorted) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= n) return;
  const float s = sigma[c];
  int rank = 0;
  for (int j = 0; j < n; ++j) {
    const float o = sigma[j];
    rank += (o > s) || (o == s && j < c);
  }
  order[rank] = c;
  if (sigma_sorted != nullptr) sigma_sorted[rank] = s;
}

// Writes the factors of one matrix in the library's layouts.  U part: u_i = a_{c_i} / sigma_i (length D);
// V part: sigma_i * V[c_i, :] (length n).  u_out is [r, D] (row i = u_i) when u_rows, else [D, r];
// v_out is [n, r] (column i) when v_cols, else [r, n].
template <typename T>
__global__ void proxy_emit_kernel(const float* __restrict__ A, const float* __restrict__ V,
                                  const float* __restrict__ sigma, const int32_t* __restrict__ order, int n, int m,
                                  int r, int u_rows, int v_cols, T* __restrict__ u_out, T* __restrict__ v_out) {
  const int i = blockIdx.x;            // 0 .. r-1
  const int c = order[i];
  const float sg = sigma[c];
  const float inv = sg > 0.f ? 1.0f / sg : 0.f;
  for (int d = threadIdx.x; d < m; d += blockDim.x) {
    const T v = from_f32<T>(A[(size_t)c * m + d] * inv);
    if (u_rows) u_out[(size_t)i * m + d] = v;
    else u_out[(size_t)d * r + i] = v;
  }
  for (int x = threadIdx.x; x < n; x += blockDim.x) {
    const T v = from_f32<T>(V[(size_t)c * n + x] * sg);
    if (v_cols) v_out[(size_t)x * r + i] = v;
    else v_out[(size_t)i * n + x] = v;
  }
}

}  // namespace

spts_status launch_proxy_importance(spts_ctx* ctx, const float* zt, int ld, int n_cal, int k, int n_channels,
                                    float* importance) {
  proxy_importance_kernel<<<n_channels, IMP_THREADS, 0, ctx->stream>>>(zt, ld, n_cal, k, importance);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

// Factorises one reduced matrix.  A [n, m], V [n, n], sigma [n], order [n] are fp32 / int32 scratch.
spts_status launch_proxy_factor(spts_ctx* ctx, const void* W, const int32_t* channels, int down, int sweeps,
                                float* A, float* V, float* sigma, int32_t* order, unsigned int* offdiag, int r,
                                void* u_out, void* v_out, float* sigma_sorted) {
  const auto& d = ctx->desc;
  const int n = d.ltp_dlow, m = d.hidden;
  cudaStream_t st = ctx->stream;
  if (d.dtype == SPTS_BF16)
    proxy_slice_kernel<bf16><<<n, 256, 0, st>>>((const bf16*)W, channels, n, m, d.ffn_dim, down, A, V);
  else
    proxy_slice_kernel<float><<<n, 256, 0, st>>>((const float*)W, channels, n, m, d.ffn_dim, down, A, V);
  SPTS_CUDA_OK(ctx);
  if (cudaMemsetAsync(offdiag, 0, sizeof(unsigned int) * (size_t)sweeps, st) != cudaSuccess) return SPTS_ERR_CUDA;
  for (int sw = 0; sw < sweeps; ++sw) {
    for (int round = 0; round < n - 1; ++round) {
      proxy_jacobi_round_kernel<<<n / 2, JAC_THREADS, 0, st>>>(A, V, n, m, round, offdiag + sw);
      SPTS_CUDA_OK(ctx);
    }
  }
  proxy_sigma_kernel<<<n, JAC_THREADS, 0, st>>>(A, m, sigma);
  SPTS_CUDA_OK(ctx);
  proxy_rank_kernel<<<ceil_div(n, 128), 128, 0, st>>>(sigma, n, order, sigma_sorted);
  SPTS_CUDA_OK(ctx);
  const int u_rows = down ? 0 : 1, v_cols = down ? 0 : 1;
  if (d.dtype == SPTS_BF16)
    proxy_emit_kernel<bf16><<<r, 256, 0, st>>>(A, V, sigma, order, n, m, r, u_rows, v_cols, (bf16*)u_out, (bf16*)v_out);
  else
    proxy_emit_kernel<float><<<r, 256, 0, st>>>(A, V, sigma, order, n, m, r, u_rows, v_cols, (float*)u_out, (float*)v_out);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

}  // namespace spts
