// Decode step (Algorithm 1 outside the prefill phase): one new token runs every layer densely
// against that layer's compressed KV cache plus itself.  Batch-1 decode streams every weight and
// every cached key / value once, so everything here is HBM-bound; the kernels are built to keep
// many 16-byte loads in flight per thread:
//
//   gemv core    one CTA = 8 weight rows (16 for the gate / up pair); its 8 warps split K, every
//                lane issues the loads of all rows of a K-chunk together, partial dots meet in
//                shared memory.  RMSNorm is an fp32 scale computed from the same pass over x.
//   epilogues    q / k / v projection with rotary embedding and the cache append fused in;
//                SwiGLU of the gate / up pair; residual update (O and down projections).
//   attention    one CTA = one KV head x one slice of the cache, serving the whole GQA group of
//                query heads at once (each cached row is read once), online softmax, then a
//                combine kernel over the slices.  bf16 caches: warp-level tensor-core MMAs with
//                both operands loaded from global memory in fragment order (dec_attn_mma_kernel);
//                fp32 caches: CUDA cores (dec_attn_partial_kernel).
//   launches     every kernel of a step is a programmatic dependent of the one before: it lets
//                its successor start, pulls what does not depend on its predecessor (weights,
//                old cache rows) towards L2 or into registers, and only then waits.
// The residual vector lives in fp32 scratch and is rounded through the storage type at the same
// points as the prefill path.
#include <type_traits>

#include "spts_common.cuh"

namespace spts {

namespace {

template <typename T> struct DV;
template <> struct DV<float> { static constexpr int N = 4; };
template <> struct DV<bf16> { static constexpr int N = 8; };

template <typename T> __device__ __forceinline__ void ld16(const T* p, float* out);
template <> __device__ __forceinline__ void ld16<float>(const float* p, float* out) {
  float4 v = __ldg(reinterpret_cast<const float4*>(p));
  out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
template <> __device__ __forceinline__ void ld16<bf16>(const bf16* p, float* out) {
  uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out[2 * i] = __uint_as_float(w[i] << 16);
    out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

// The same, read at L2 (ld.global.cg): for data written by the kernel just before this one.  Kernels of a chain of
// programmatic dependents overlap, so an L1 line of this SM may be older than the predecessor's write.
template <typename T> __device__ __forceinline__ void ld16_cg(const T* p, float* out);
template <> __device__ __forceinline__ void ld16_cg<float>(const float* p, float* out) {
  float4 v = __ldcg(reinterpret_cast<const float4*>(p));
  out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
template <> __device__ __forceinline__ void ld16_cg<bf16>(const bf16* p, float* out) {
  uint4 v = __ldcg(reinterpret_cast<const uint4*>(p));
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

constexpr int GV_THREADS = 256;   // 8 warps
constexpr int GV_WARPS = 8;

// dots[r] = sum_k x[k] * row_r[k] for R rows given by pointer, and sumsq = sum_k x[k]^2.
// Results are valid in shared memory (dots_out[0..R), *ss_out) for all threads after the call.
template <typename T, int R>
__device__ __forceinline__ void gemv_rows(const T* (&rowp)[R], int K, const float* __restrict__ x,
                                          float* dots_out, float* ss_out) {
  constexpr int V = DV<T>::N;
  __shared__ float red[GV_WARPS][R + 1];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float acc[R];
#pragma unroll
  for (int r = 0; r < R; ++r) acc[r] = 0.f;
  float ss = 0.f;
  const int c0 = (warp * 32 + lane) * V;
  dep_launch();
  // The weights do not depend on the previous kernel: the block's rows are pulled towards L2 while it finishes,
  // one bulk prefetch per 8 KiB piece of a row (far fewer requests than a prefetch per 16-byte chunk, and measured
  // twice as effective on the step time).  Rows are 16-byte multiples (K is a multiple of 8 elements).
  {
    constexpr int PIECE = 8192;
    const int row_bytes = K * (int)sizeof(T);
    const int npiece = (row_bytes + PIECE - 1) / PIECE;
    for (int u = threadIdx.x; u < R * npiece; u += GV_THREADS) {
      const int r = u / npiece, pc = u - r * npiece;
      const int bytes = min(PIECE, row_bytes - pc * PIECE) & ~15;
      const char* src = nullptr;
#pragma unroll
      for (int rr = 0; rr < R; ++rr)
        if (rr == r) src = reinterpret_cast<const char*>(rowp[rr]) + (size_t)pc * PIECE;
      if (bytes > 0) asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
    }
  }
  dep_wait();                                                    // x does depend on it
  for (int c = c0; c < K; c += GV_THREADS * V) {
    float w[R][V];
#pragma unroll
    for (int r = 0; r < R; ++r) ld16<T>(rowp[r] + c, w[r]);      // R independent 16-byte loads in flight
    float xv[V];
#pragma unroll
    for (int e = 0; e < V; e += 4) {
      float4 t = __ldcg(reinterpret_cast<const float4*>(x + c + e));   // x comes from the previous kernel: read at L2
      xv[e] = t.x; xv[e + 1] = t.y; xv[e + 2] = t.z; xv[e + 3] = t.w;
    }
#pragma unroll
    for (int e = 0; e < V; ++e) {
      ss = fmaf(xv[e], xv[e], ss);
#pragma unroll
      for (int r = 0; r < R; ++r) acc[r] = fmaf(xv[e], w[r][e], acc[r]);
    }
  }
#pragma unroll
  for (int r = 0; r < R; ++r) acc[r] = warp_sum(acc[r]);
  ss = warp_sum(ss);
  if (lane == 0) {
#pragma unroll
    for (int r = 0; r < R; ++r) red[warp][r] = acc[r];
    red[warp][R] = ss;
  }
  __syncthreads();
  if (threadIdx.x <= R) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < GV_WARPS; ++w) s += red[w][threadIdx.x];
    if (threadIdx.x < R) dots_out[threadIdx.x] = s;
    else *ss_out = s;
  }
  __syncthreads();
}

// out[j] = round(out[j] + x . W[j, :])   (O and down projections: residual update, Eq. 2 with all rows)
template <typename T>
__global__ void __launch_bounds__(GV_THREADS)
gemv_resid_kernel(const T* __restrict__ W, int rows, int K, const float* __restrict__ x, float* __restrict__ out) {
  __shared__ float dots[8];
  __shared__ float ss;
  const int r0 = blockIdx.x * 8;
  const T* rowp[8];
#pragma unroll
  for (int r = 0; r < 8; ++r) rowp[r] = W + (size_t)min(r0 + r, rows - 1) * K;
  gemv_rows<T, 8>(rowp, K, x, dots, &ss);
  if (threadIdx.x < 8 && r0 + threadIdx.x < rows) {
    const int j = r0 + threadIdx.x;
    out[j] = round_through<T>(__ldcg(&out[j]) + dots[threadIdx.x]);
  }
}

// hm[j] = round(silu(rs * x . Wg[j, :]) * (rs * x . Wu[j, :])),  rs = 1 / sqrt(mean(x^2) + eps)   (Eq. 6)
// One CTA = four gate rows and the same four up rows (eight streams, like the other kernels, so that four CTAs
// fit on an SM).
template <typename T>
__global__ void __launch_bounds__(GV_THREADS)
gemv_swiglu_kernel(const T* __restrict__ Wg, const T* __restrict__ Wu, int rows, int K, const float* __restrict__ x,
                   float eps, float* __restrict__ hm) {
  __shared__ float dots[8];
  __shared__ float ss;
  const int r0 = blockIdx.x * 4;
  const T* rowp[8];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const size_t off = (size_t)min(r0 + r, rows - 1) * K;
    rowp[r] = Wg + off;
    rowp[4 + r] = Wu + off;
  }
  gemv_rows<T, 8>(rowp, K, x, dots, &ss);
  if (threadIdx.x < 4 && r0 + threadIdx.x < rows) {
    const float rs = 1.0f / sqrtf(ss / (float)K + eps);
    const float g = dots[threadIdx.x] * rs, u = dots[4 + threadIdx.x] * rs;
    hm[r0 + threadIdx.x] = round_through<T>(g / (1.0f + expf(-g)) * u);
  }
}

// logits[j] = rs * x . W[j, :]   (first-token head)
template <typename T>
__global__ void __launch_bounds__(GV_THREADS)
gemv_norm_kernel(const T* __restrict__ W, int rows, int K, const float* __restrict__ x, float eps,
                 float* __restrict__ out) {
  __shared__ float dots[8];
  __shared__ float ss;
  const int r0 = blockIdx.x * 8;
  const T* rowp[8];
#pragma unroll
  for (int r = 0; r < 8; ++r) rowp[r] = W + (size_t)min(r0 + r, rows - 1) * K;
  gemv_rows<T, 8>(rowp, K, x, dots, &ss);
  if (threadIdx.x < 8 && r0 + threadIdx.x < rows)
    out[r0 + threadIdx.x] = dots[threadIdx.x] * (1.0f / sqrtf(ss / (float)K + eps));
}

// q, k, v projections of the new token with RMSNorm scale, rotary embedding (q, k) and the cache
// append fused in.  Blocks [0, nq) serve q, [nq, nq + nk) k -- eight rows each: four rotary pairs
// (i, i + d/2) of one head -- and the rest v, eight consecutive rows.
template <typename T>
__global__ void __launch_bounds__(GV_THREADS)
dec_qkv_kernel(const T* __restrict__ wq, const T* __restrict__ wk, const T* __restrict__ wv, int H, int Hkv, int d,
               int K, const float* __restrict__ x, float eps, int pos, double theta, float* __restrict__ q32,
               T* __restrict__ kc, T* __restrict__ vc, int32_t* __restrict__ pc, int slot) {
  __shared__ float dots[8];
  __shared__ float ss;
  const int half = d >> 1;
  const int per_head = half / 4;                     // blocks per head for q and k
  const int nq = H * per_head, nk = Hkv * per_head;
  const int b = blockIdx.x;
  const T* rowp[8];
  int kind, h = 0, i0 = 0, v0 = 0;                   // kind 0 q, 1 k, 2 v
  if (b < nq + nk) {
    kind = b < nq ? 0 : 1;
    const int bb = kind == 0 ? b : b - nq;
    h = bb / per_head;
    i0 = (bb - h * per_head) * 4;
    const T* w = kind == 0 ? wq : wk;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      rowp[r] = w + (size_t)(h * d + i0 + r) * K;
      rowp[4 + r] = w + (size_t)(h * d + half + i0 + r) * K;
    }
  } else {
    kind = 2;
    v0 = (b - nq - nk) * 8;
#pragma unroll
    for (int r = 0; r < 8; ++r) rowp[r] = wv + (size_t)min(v0 + r, Hkv * d - 1) * K;
  }
  // the rotary factors depend on the position only: the (slow) double-precision evaluation runs while the
  // previous kernel is still finishing, ahead of the dependency wait inside gemv_rows
  const int t = threadIdx.x;
  float cf = 1.f, sf = 0.f;
  if (kind != 2 && t < 4) {
    const double inv = exp2(-(double)(2 * (i0 + t)) / (double)d * log2(theta));
    double sn, cs;
    sincos((double)pos * inv, &sn, &cs);
    cf = (float)cs; sf = (float)sn;
  }
  gemv_rows<T, 8>(rowp, K, x, dots, &ss);
  const float rs = 1.0f / sqrtf(ss / (float)K + eps);
  if (kind == 2) {
    if (t < 8 && v0 + t < Hkv * d) vc[(size_t)slot * Hkv * d + v0 + t] = from_f32<T>(dots[t] * rs);
    return;
  }
  if (t < 4) {
    const int i = i0 + t;
    const float a = dots[t] * rs, bb2 = dots[4 + t] * rs;
    const float r1 = a * cf - bb2 * sf, r2 = bb2 * cf + a * sf;
    if (kind == 0) {
      q32[h * d + i] = round_through<T>(r1);
      q32[h * d + i + half] = round_through<T>(r2);
    } else {
      kc[((size_t)slot * Hkv + h) * d + i] = from_f32<T>(r1);
      kc[((size_t)slot * Hkv + h) * d + i + half] = from_f32<T>(r2);
    }
  }
  if (b == 0 && t == 32) pc[slot] = pos;
}

// Split-KV attention of the new token.  Block (x, s): query heads [x * G, x * G + G) -- all of
// them read KV head (x * G) / group -- over cached rows [s * len / ns, (s + 1) * len / ns).
// A cached row is D * sizeof(T) bytes = LPK lanes x 16 bytes, so a warp takes 32 / LPK rows per
// step and two steps are in flight.  part[(h * ns + s)] = (max, sum, o[D]) per query head.
template <typename T, int D, int G>
__global__ void __launch_bounds__(128)
dec_attn_partial_kernel(const float* __restrict__ q32, const T* __restrict__ kc, const T* __restrict__ vc, int len,
                        int H, int Hkv, int nsplit, float* __restrict__ part) {
  constexpr int V = DV<T>::N;              // elements per 16-byte chunk
  constexpr int LPK = D / V;               // lanes per cached row
  constexpr int KPW = 32 / LPK;            // rows per warp step
  constexpr int NP = 4 * KPW;              // partial states per block
  __shared__ float sm_m[NP][G], sm_l[NP][G];
  __shared__ float sm_o[NP][G][D];
  dep_launch();
  dep_wait();                                        // q and the cache's newest row come from the previous kernel
  const int hb = blockIdx.x * G, s = blockIdx.y;
  const int kvh = hb / (H / Hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPK, li = lane % LPK;       // which row of the step, which chunk of the row
  const int j0 = (int)((long)len * s / nsplit), j1 = (int)((long)len * (s + 1) / nsplit);
  const float scale = rsqrtf((float)D);
  float q[G][V], o[G][V], m[G], l[G];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m[g] = -INFINITY; l[g] = 0.f;
#pragma unroll
    for (int e = 0; e < V; ++e) { q[g][e] = __ldcg(&q32[(hb + g) * D + li * V + e]) * scale; o[g][e] = 0.f; }
  }
  const size_t rstride = (size_t)Hkv * D;
  const T* kbase = kc + (size_t)kvh * D + li * V;
  const T* vbase = vc + (size_t)kvh * D + li * V;
  constexpr int STEP = 4 * KPW;                      // rows per block step
  // the trip count is the same for every lane of a warp (the shuffles below need all of them)
  for (int jw = j0 + warp * KPW; jw < j1; jw += 2 * STEP) {
    const int ja = jw + sub, jb = ja + STEP;
    const bool hasa = ja < j1, hasb = jb < j1;
    float ka[V], va[V], kb[V], vb[V];
    ld16_cg<T>(kbase + (size_t)(hasa ? ja : j0) * rstride, ka);      // the newest row is the previous kernel's
    ld16_cg<T>(vbase + (size_t)(hasa ? ja : j0) * rstride, va);
    ld16_cg<T>(kbase + (size_t)(hasb ? jb : j0) * rstride, kb);
    ld16_cg<T>(vbase + (size_t)(hasb ? jb : j0) * rstride, vb);
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float da = 0.f, db = 0.f;
#pragma unroll
      for (int e = 0; e < V; ++e) { da = fmaf(q[g][e], ka[e], da); db = fmaf(q[g][e], kb[e], db); }
#pragma unroll
      for (int off = LPK / 2; off > 0; off >>= 1) {
        da += __shfl_xor_sync(0xffffffffu, da, off);
        db += __shfl_xor_sync(0xffffffffu, db, off);
      }
      if (hasa) {                                      // hasb implies hasa
        if (!hasb) db = -INFINITY;
        const float mn = fmaxf(m[g], fmaxf(da, db));
        const float corr = expf(m[g] - mn), pa = expf(da - mn), pb = expf(db - mn);
        l[g] = l[g] * corr + pa + pb;
#pragma unroll
        for (int e = 0; e < V; ++e) o[g][e] = fmaf(pa, va[e], fmaf(pb, vb[e], o[g][e] * corr));
        m[g] = mn;
      }
    }
  }
  const int pi = warp * KPW + sub;
#pragma unroll
  for (int g = 0; g < G; ++g) {
    if (li == 0) { sm_m[pi][g] = m[g]; sm_l[pi][g] = l[g]; }
#pragma unroll
    for (int e = 0; e < V; ++e) sm_o[pi][g][li * V + e] = o[g][e];
  }
  __syncthreads();
  for (int t = threadIdx.x; t < G * D; t += 128) {
    const int g = t / D, c = t - g * D;
    float M = -INFINITY;
#pragma unroll
    for (int p = 0; p < NP; ++p) M = fmaxf(M, sm_m[p][g]);
    float L = 0.f, acc = 0.f;
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const float f = sm_m[p][g] == -INFINITY ? 0.f : expf(sm_m[p][g] - M);
      L += sm_l[p][g] * f;
      acc = fmaf(sm_o[p][g][c], f, acc);
    }
    float* pp = part + ((size_t)(hb + g) * nsplit + s) * (D + 2);
    if (c == 0) { pp[0] = M; pp[1] = L; }
    pp[2 + c] = acc;
  }
}

// ---- the same partial attention for bf16 caches, on mma.sync (m16n8k16, fp32 accumulation) ----
// The CUDA-core kernel above spends ~80 warp instructions per cached row (dot products spread over 16 lanes,
// shuffles, exponentials repeated in every lane); here a warp takes 16 cached rows per step with 32 MMAs:
//   S[q, row] = Q K^T   M = up to 16 query heads of the GQA group (rows past the group are zero), N = 8 rows, K = d
//   O[q, dim] += P V    M = the same queries, N = 8 dims, K = 16 rows
// Both operands come straight from global memory in 16-byte loads, with no shared-memory staging: a dot product
// does not care about the order of its terms, so the k index of the first product and the n index of the second
// are permuted to whatever order the loads deliver.
//   K:  lane (g, c) = (lane / 4, lane % 4) loads, of row r0 + 8u + g, the 8 elements 32j + 8c .. + 7 (j = 0 .. d/32 - 1);
//       elements 4h .. 4h + 3 of that chunk are the lane's share of k-step 2j + h, and Q's fragment is built with
//       the same map.
//   V:  lane (g, c) loads, of rows r0 + 2c, r0 + 2c + 1, r0 + 8 + 2c, r0 + 9 + 2c, the 8 elements 64x + 8g .. + 7
//       (x = 0 .. d/64 - 1; the eight lanes of a row read 128 contiguous bytes per load); n-tile v = 8x + e then
//       holds dims {64x + 8g + e}, and byte permutes pair the two rows of a k index.
// S's accumulator fragment is P's A fragment (rows 2c, 2c + 1 of n-tile u = k indices 2c + 8u, 2c + 8u + 1).
// O is rescaled only in steps where some query's running maximum moved.
__device__ __forceinline__ void mma_bf16_16816(float& d0, float& d1, float& d2, float& d3, uint32_t a0, uint32_t a1,
                                               uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1, float c0, float c1,
                                               float c2, float c3) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
               : "=f"(d0), "=f"(d1), "=f"(d2), "=f"(d3)
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(c0), "f"(c1), "f"(c2), "f"(c3));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// HI: the block serves more than 8 query heads (fragment rows 8..15 carry heads too).
template <int D, bool HI>
__global__ void __launch_bounds__(128, 3)
dec_attn_mma_kernel(const float* __restrict__ q32, const bf16* __restrict__ kc, const bf16* __restrict__ vc, int len,
                    int H, int Hkv, int nsplit, float* __restrict__ part) {
  constexpr int NJ = D / 32;               // 16-byte chunks of a K row per lane
  constexpr int NT = D / 16;               // k-steps of Q K^T
  constexpr int NV = D / 8;                // n-tiles of P V = elements of a V row per lane
  constexpr int VQ = NV / 8;               // 16-byte chunks of a V row per lane
  constexpr int NQ = HI ? 16 : 8;
  __shared__ float sm_m[4][NQ], sm_l[4][NQ];
  // a lane's accumulators are, per x, the 16 dims 64x + 16c .. + 15: stored as [query][c][x][16] with four floats of
  // padding per (query, c), the 16-byte stores of a quarter warp fall into distinct banks
  constexpr int OC = 16 * VQ + 4;
  __shared__ __align__(16) float sm_o[4][NQ][4][OC];
  dep_launch();
  const int G = H / Hkv, qb = (G + 15) / 16;
  const int kvh = blockIdx.x / qb, qoff = (blockIdx.x % qb) * 16, s = blockIdx.y;
  const int hb = kvh * G + qoff, nq = min(16, G - qoff);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;
  const int j0 = (int)((long)len * s / nsplit), j1 = (int)((long)len * (s + 1) / nsplit);
  const float sl = rsqrtf((float)D) * 1.4426950408889634f;

  float o[NV][HI ? 4 : 2];
#pragma unroll
  for (int v = 0; v < NV; ++v)
#pragma unroll
    for (int i = 0; i < (HI ? 4 : 2); ++i) o[v][i] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

  const size_t rstride = (size_t)Hkv * D;
  const bf16* kbase = kc + (size_t)kvh * D + 8 * c;
  const bf16* vbase = vc + (size_t)kvh * D + g * 8;
  // Only q and the cache's newest row (index len - 1) come from the previous kernel.  Ahead of the dependency
  // wait the warp loads its first 16 rows into registers -- unless they reach the newest row -- and pulls its
  // later rows towards L2, so that the cache streams in while the projection kernel is still running.
  uint4 kq[2][NJ], vq[4][VQ];
  auto load_rows = [&](int r0) {
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const bf16* kp = kbase + (size_t)min(r0 + 8 * u + g, j1 - 1) * rstride;
#pragma unroll
      for (int j = 0; j < NJ; ++j) kq[u][j] = __ldcg(reinterpret_cast<const uint4*>(kp + 32 * j));
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const bf16* vp = vbase + (size_t)min(r0 + 8 * (i >> 1) + 2 * c + (i & 1), j1 - 1) * rstride;
#pragma unroll
      for (int x = 0; x < VQ; ++x) vq[i][x] = __ldcg(reinterpret_cast<const uint4*>(vp + 64 * x));
    }
  };
  const int r_first = j0 + warp * 16;
  bool loaded = false;
  if (r_first < j1 && r_first + 16 <= len - 1) { load_rows(r_first); loaded = true; }
  for (int r0 = r_first + (loaded ? 64 : 0); r0 < j1; r0 += 64) {
    // 16 rows x (D * 2) bytes of K and of V = 128-byte lines, spread over the lanes
    for (int ln = lane; ln < 16 * (D * 2 / 128); ln += 32) {
      const int row = min(r0 + ln / (D * 2 / 128), j1 - 1);
      const size_t off = ((size_t)row * Hkv + kvh) * D + (ln % (D * 2 / 128)) * 64;
      asm volatile("prefetch.global.L2 [%0];" ::"l"(kc + off));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(vc + off));
    }
  }
  dep_wait();
  uint32_t qa[NT][HI ? 4 : 2];
#pragma unroll
  for (int t = 0; t < NT; ++t) {
    const int e = 32 * (t >> 1) + 8 * c + 4 * (t & 1);
    float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
    if (g < nq) lo = __ldcg(reinterpret_cast<const float4*>(q32 + (size_t)(hb + g) * D + e));
    qa[t][0] = pack_bf16x2(lo.x, lo.y);
    qa[t][1] = pack_bf16x2(lo.z, lo.w);
    if (HI) {
      if (g + 8 < nq) hi = __ldcg(reinterpret_cast<const float4*>(q32 + (size_t)(hb + g + 8) * D + e));
      qa[t][2] = pack_bf16x2(hi.x, hi.y);
      qa[t][3] = pack_bf16x2(hi.z, hi.w);
    }
  }
  for (int r0 = r_first; r0 < j1; r0 += 64) {       // the same trip count for every lane of a warp
    if (!loaded) load_rows(r0);
    loaded = false;
    // S = Q K^T for the two 8-row tiles
    float sc[2][4];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      sc[u][0] = sc[u][1] = sc[u][2] = sc[u][3] = 0.f;
#pragma unroll
      for (int t = 0; t < NT; ++t) {
        const uint4 kk = kq[u][t >> 1];
        const uint32_t b0 = (t & 1) ? kk.z : kk.x, b1 = (t & 1) ? kk.w : kk.y;
        mma_bf16_16816(sc[u][0], sc[u][1], sc[u][2], sc[u][3], qa[t][0], HI ? qa[t][2] : 0u, qa[t][1],
                       HI ? qa[t][3] : 0u, b0, b1, sc[u][0], sc[u][1], sc[u][2], sc[u][3]);
      }
      // rows past the slice
      const int ra = r0 + 8 * u + 2 * c;
      if (ra >= j1) { sc[u][0] = -INFINITY; sc[u][2] = -INFINITY; }
      if (ra + 1 >= j1) { sc[u][1] = -INFINITY; sc[u][3] = -INFINITY; }
    }
    float x0 = fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1]));
    x0 = fmaxf(x0, __shfl_xor_sync(0xffffffffu, x0, 1));
    x0 = fmaxf(x0, __shfl_xor_sync(0xffffffffu, x0, 2));
    float x1 = -INFINITY;
    if (HI) {
      x1 = fmaxf(fmaxf(sc[0][2], sc[0][3]), fmaxf(sc[1][2], sc[1][3]));
      x1 = fmaxf(x1, __shfl_xor_sync(0xffffffffu, x1, 1));
      x1 = fmaxf(x1, __shfl_xor_sync(0xffffffffu, x1, 2));
    }
    const bool moved = x0 > m0 || (HI && x1 > m1);
    if (__any_sync(0xffffffffu, moved)) {
      const float n0 = fmaxf(m0, x0), n1 = fmaxf(m1, x1);
      const float c0 = exp2f((m0 - n0) * sl), c1 = HI ? exp2f((m1 - n1) * sl) : 0.f;   // first step: exp2(-inf) = 0
      m0 = n0; l0 *= c0;
      if (HI) { m1 = n1; l1 *= c1; }
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        o[v][0] *= c0; o[v][1] *= c0;
        if (HI) { o[v][2] *= c1; o[v][3] *= c1; }
      }
    }
    uint32_t pa[4];
    {
      const float b0 = m0 * sl;
      const float p00 = exp2f(fmaf(sc[0][0], sl, -b0)), p01 = exp2f(fmaf(sc[0][1], sl, -b0));
      const float p10 = exp2f(fmaf(sc[1][0], sl, -b0)), p11 = exp2f(fmaf(sc[1][1], sl, -b0));
      l0 += (p00 + p01) + (p10 + p11);
      pa[0] = pack_bf16x2(p00, p01); pa[2] = pack_bf16x2(p10, p11);
      pa[1] = 0u; pa[3] = 0u;
      if (HI) {
        const float b1 = m1 * sl;
        const float q00 = exp2f(fmaf(sc[0][2], sl, -b1)), q01 = exp2f(fmaf(sc[0][3], sl, -b1));
        const float q10 = exp2f(fmaf(sc[1][2], sl, -b1)), q11 = exp2f(fmaf(sc[1][3], sl, -b1));
        l1 += (q00 + q01) + (q10 + q11);
        pa[1] = pack_bf16x2(q00, q01); pa[3] = pack_bf16x2(q10, q11);
      }
    }
    // O += P V
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const int x = v >> 3, w = (v >> 1) & 3;
      const uint32_t r00 = (&vq[0][x].x)[w], r01 = (&vq[1][x].x)[w], r10 = (&vq[2][x].x)[w], r11 = (&vq[3][x].x)[w];
      const uint32_t sel = (v & 1) ? 0x7632u : 0x5410u;
      const uint32_t b0 = __byte_perm(r00, r01, sel), b1 = __byte_perm(r10, r11, sel);
      if (HI) {
        mma_bf16_16816(o[v][0], o[v][1], o[v][2], o[v][3], pa[0], pa[1], pa[2], pa[3], b0, b1, o[v][0], o[v][1],
                       o[v][2], o[v][3]);
      } else {
        float d2, d3;
        mma_bf16_16816(o[v][0], o[v][1], d2, d3, pa[0], 0u, pa[2], 0u, b0, b1, o[v][0], o[v][1], 0.f, 0.f);
      }
    }
  }
  // the four lanes of a query hold partial sums of l
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  if (HI) {
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  }
  if (c == 0) {
    sm_m[warp][g] = m0; sm_l[warp][g] = l0;
    if (HI) { sm_m[warp][g + 8] = m1; sm_l[warp][g + 8] = l1; }
  }
  // accumulator columns 2c, 2c + 1 of n-tile 8x + e are dims 64x + 16c + e and 64x + 16c + 8 + e
#pragma unroll
  for (int x = 0; x < VQ; ++x)
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int e4 = 0; e4 < 2; ++e4) {
        const int v = 8 * x + 4 * e4;
        *reinterpret_cast<float4*>(&sm_o[warp][g][c][16 * x + 8 * i + 4 * e4]) =
            make_float4(o[v][i], o[v + 1][i], o[v + 2][i], o[v + 3][i]);
        if (HI)
          *reinterpret_cast<float4*>(&sm_o[warp][g + 8][c][16 * x + 8 * i + 4 * e4]) =
              make_float4(o[v][2 + i], o[v + 1][2 + i], o[v + 2][2 + i], o[v + 3][2 + i]);
      }
  __syncthreads();
  const float scale = rsqrtf((float)D);
  for (int t = threadIdx.x; t < nq * D; t += 128) {
    const int q = t / D, dim = t - q * D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < 4; ++w) M = fmaxf(M, sm_m[w][q]);
    float L = 0.f, acc = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float f = sm_m[w][q] == -INFINITY ? 0.f : exp2f((sm_m[w][q] - M) * sl);
      L += sm_l[w][q] * f;
      acc = fmaf(sm_o[w][q][(dim >> 4) & 3][16 * (dim >> 6) + (dim & 15)], f, acc);
    }
    float* pp = part + ((size_t)(hb + q) * nsplit + s) * (D + 2);
    if (dim == 0) { pp[0] = M * scale; pp[1] = L; }
    pp[2 + dim] = acc;
  }
}

constexpr int DEC_MAX_SPLIT = 64;

// Combines the slices of one query head.  Thread s < nsplit takes slice s's (max, sum), so the global maximum and
// the weights exp(max_s - M) come from one parallel step; then the block's 512 / d thread groups each sum one
// dimension per thread over every (512 / d)-th slice, all of a group's loads in flight together, and the groups
// meet in shared memory.  d divides 512, nsplit <= 64.
template <typename T>
__global__ void __launch_bounds__(512)
dec_attn_combine_kernel(const float* __restrict__ part, int nsplit, int d, float* __restrict__ att32) {
  __shared__ float f[DEC_MAX_SPLIT];
  __shared__ float red[4];
  __shared__ float accs[512];
  dep_launch();
  dep_wait();
  const int h = blockIdx.x, t = threadIdx.x;
  const float* ph = part + (size_t)h * nsplit * (d + 2);
  float m = -INFINITY, l = 0.f;
  if (t < nsplit) {
    m = __ldcg(&ph[(size_t)t * (d + 2)]);
    l = __ldcg(&ph[(size_t)t * (d + 2) + 1]);
  }
  float v = warp_max(m);
  if (t < 64 && (t & 31) == 0) red[t >> 5] = v;
  __syncthreads();
  const float M = fmaxf(red[0], red[1]);
  const float fs = m == -INFINITY ? 0.f : expf(m - M);
  if (t < nsplit) f[t] = fs;
  v = warp_sum(l * fs);
  if (t < 64 && (t & 31) == 0) red[2 + (t >> 5)] = v;
  __syncthreads();
  const float L = red[2] + red[3];
  const int ngrp = 512 / d, grp = t / d, dim = t - grp * d;
  constexpr int U = 16;
  float acc = 0.f;
  for (int s0 = grp; s0 < nsplit; s0 += ngrp * U) {
    float x[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int s = s0 + u * ngrp;
      x[u] = s < nsplit ? __ldcg(&ph[(size_t)s * (d + 2) + 2 + dim]) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int s = s0 + u * ngrp;
      if (s < nsplit) acc = fmaf(x[u], f[s], acc);
    }
  }
  accs[t] = acc;
  __syncthreads();
  if (t < d) {
    float a = 0.f;
    for (int gq = 0; gq < ngrp; ++gq) a += accs[gq * d + t];
    att32[h * d + t] = round_through<T>(a / L);
  }
}

#define LAUNCH_DEP(ctx, ...)                                                      \
  do {                                                                            \
    if (launch_dependent(__VA_ARGS__) != cudaSuccess) return SPTS_ERR_CUDA;       \
    (ctx)->launches++;                                                            \
  } while (0)
#define TRY_DEC(...) do { spts_status s__ = (__VA_ARGS__); if (s__ != SPTS_OK) return s__; } while (0)

template <typename T, int D>
spts_status launch_attn_partial(spts_ctx* ctx, const float* q32, const spts_kv_layer* cache, int len, int nsplit,
                                float* part) {
  const auto& d = ctx->desc;
  const int H = d.n_q_heads, Hkv = d.n_kv_heads, group = H / Hkv;
  cudaStream_t st = ctx->stream;
  const T* kc = (const T*)cache->k;
  const T* vc = (const T*)cache->v;
  if constexpr (std::is_same<T, bf16>::value) {
    const dim3 grid(Hkv * ceil_div(group, 16), nsplit);
    if (group > 8)
      LAUNCH_DEP(ctx, dec_attn_mma_kernel<D, true>, grid, dim3(128), st, q32, kc, vc, len, H, Hkv, nsplit, part);
    else
      LAUNCH_DEP(ctx, dec_attn_mma_kernel<D, false>, grid, dim3(128), st, q32, kc, vc, len, H, Hkv, nsplit, part);
    return SPTS_OK;
  }
  // all query heads of a GQA group in one block when the group size is 2, 4 or 8; else one head per block
  if (group % 8 == 0)
    LAUNCH_DEP(ctx, dec_attn_partial_kernel<T, D, 8>, dim3(H / 8, nsplit), dim3(128), st, q32, kc, vc, len, H, Hkv, nsplit, part);
  else if (group % 4 == 0)
    LAUNCH_DEP(ctx, dec_attn_partial_kernel<T, D, 4>, dim3(H / 4, nsplit), dim3(128), st, q32, kc, vc, len, H, Hkv, nsplit, part);
  else if (group % 2 == 0)
    LAUNCH_DEP(ctx, dec_attn_partial_kernel<T, D, 2>, dim3(H / 2, nsplit), dim3(128), st, q32, kc, vc, len, H, Hkv, nsplit, part);
  else
    LAUNCH_DEP(ctx, dec_attn_partial_kernel<T, D, 1>, dim3(H, nsplit), dim3(128), st, q32, kc, vc, len, H, Hkv, nsplit, part);
  return SPTS_OK;
}

template <typename T>
spts_status decode_layer_t(spts_ctx* ctx, const spts_layer_weights* w, spts_kv_layer* cache, float* x32,
                           int32_t pos) {
  const auto& d = ctx->desc;
  cudaStream_t st = ctx->stream;
  const int D = d.hidden, H = d.n_q_heads, Hkv = d.n_kv_heads, hd = d.head_dim, Dff = d.ffn_dim;
  float* base = (float*)ctx->ws.dec;
  float* q32 = base + D;                     // [H*hd]
  float* att32 = q32 + H * hd;               // [H*hd]
  float* hm32 = att32 + H * hd;              // [Dff]
  float* part = hm32 + Dff;                  // [H, DEC_MAX_SPLIT, hd + 2]
  if (cache->len + 1 > cache->capacity) return SPTS_ERR_WORKSPACE;
  const int slot = cache->len;
  const int per_head = hd / 8;
  const int qkv_blocks = (H + Hkv) * per_head + ceil_div(Hkv * hd, 8);
  LAUNCH_DEP(ctx, dec_qkv_kernel<T>, dim3(qkv_blocks), dim3(GV_THREADS), st, (const T*)w->wq, (const T*)w->wk,
             (const T*)w->wv, H, Hkv, hd, D, (const float*)x32, d.rms_eps, (int)pos, (double)d.rope_theta, q32,
             (T*)cache->k, (T*)cache->v, cache->pos, slot);
  const int len = slot + 1;                  // the host-side cache->len is advanced by the caller once the whole step is enqueued
  int nsplit = min(DEC_MAX_SPLIT, max(1, len / 128));
  if (std::is_same<T, bf16>::value)      // the tensor-core kernel holds three blocks per SM: keep the slices to one wave
    nsplit = max(1, min(nsplit, 3 * ctx->sm_count / (Hkv * ceil_div(H / Hkv, 16))));
  if (hd == 128) TRY_DEC(launch_attn_partial<T, 128>(ctx, q32, cache, len, nsplit, part));
  else TRY_DEC(launch_attn_partial<T, 64>(ctx, q32, cache, len, nsplit, part));
  LAUNCH_DEP(ctx, dec_attn_combine_kernel<T>, dim3(H), dim3(512), st, (const float*)part, nsplit, hd, att32);
  LAUNCH_DEP(ctx, gemv_resid_kernel<T>, dim3(ceil_div(D, 8)), dim3(GV_THREADS), st, (const T*)w->wo, D, H * hd,
             (const float*)att32, x32);
  LAUNCH_DEP(ctx, gemv_swiglu_kernel<T>, dim3(ceil_div(Dff, 4)), dim3(GV_THREADS), st, (const T*)w->w_gate,
             (const T*)w->w_up, Dff, D, (const float*)x32, d.rms_eps, hm32);
  LAUNCH_DEP(ctx, gemv_resid_kernel<T>, dim3(ceil_div(D, 8)), dim3(GV_THREADS), st, (const T*)w->w_down, D, Dff,
             (const float*)hm32, x32);
  return SPTS_OK;
}

}  // namespace

size_t decode_scratch_floats(const spts_model_desc& d) {
  return (size_t)d.hidden + 2 * (size_t)d.n_q_heads * d.head_dim + (size_t)d.ffn_dim +
         (size_t)d.n_q_heads * DEC_MAX_SPLIT * (d.head_dim + 2) + 64 + 2 * ARGMAX_BLOCKS;
}

// [ARGMAX_BLOCKS] values, then [ARGMAX_BLOCKS] indices: the tail of the decode scratch
float* argmax_scratch(spts_ctx* ctx) {
  return (float*)ctx->ws.dec + decode_scratch_floats(ctx->desc) - 2 * ARGMAX_BLOCKS;
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

// logits = rstd(x) * lm_head x for one hidden row held in fp32 (x32) -- shared with the first-token head
spts_status launch_head_logits(spts_ctx* ctx, const float* x32, const void* lm_head, float* logits) {
  const auto& d = ctx->desc;
  if (d.dtype == SPTS_BF16)
    gemv_norm_kernel<bf16><<<ceil_div(d.vocab, 8), GV_THREADS, 0, ctx->stream>>>((const bf16*)lm_head, d.vocab, d.hidden,
                                                                                 x32, d.rms_eps, logits);
  else
    gemv_norm_kernel<float><<<ceil_div(d.vocab, 8), GV_THREADS, 0, ctx->stream>>>((const float*)lm_head, d.vocab,
                                                                                  d.hidden, x32, d.rms_eps, logits);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

}  // namespace spts
