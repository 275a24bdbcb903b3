// Top-k selection (Eq. 5 / 15 / 16) by radix select, and the gathers used by stage-end
// compaction (Algorithm 1, "X <- X[T, :]").  Integer / compare work only: results are exact.
//
// Selection rule: score descending, then index ascending; -0.0 == +0.0; NaN ranks with -inf;
// with SPTS_FORCE_LAST the last element ranks first.  Output indices are ascending.
#include <mutex>

#include "spts_common.cuh"

namespace spts {

namespace {

constexpr int TK_THREADS = 256;
constexpr int TK_PER_THREAD = TOPK_CHUNK / TK_THREADS;  // 8

// scratch layout (uint32 words)
constexpr int SC_HIST = 0;            // [4][256]
constexpr int SC_PREFIX = 4 * 256;    // threshold key bits found so far
constexpr int SC_KREM = SC_PREFIX + 1;  // how many still to take inside the current bucket
constexpr int SC_DONE = SC_PREFIX + 2;  // blocks finished (reset by the last block)
constexpr int SC_NAN = SC_PREFIX + 3;
constexpr int SC_CTA = SC_PREFIX + 16;  // [2][TOPK_MAX_CTAS]: out_base, eq_base

__device__ __forceinline__ uint32_t score_key(float s, bool* nonfinite) {
  uint32_t u = __float_as_uint(s);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) {  // NaN ranks with -inf
    *nonfinite = true;
    return 0x007FFFFFu;
  }
  if (u == 0x80000000u) u = 0u;  // -0.0 -> +0.0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ uint32_t load_key(const float* scores, int i, int N, bool force_last,
                                             bool* nonfinite) {
  if (force_last && i == N - 1) return 0xFFFFFFFFu;
  return score_key(scores[i], nonfinite);
}

// One radix pass: histogram of the 8-bit digit at `shift` over the keys that match the prefix
// found so far; the last block to finish picks the bucket holding the k-th largest key.
__global__ void __launch_bounds__(TK_THREADS)
topk_hist_kernel(const float* __restrict__ scores, int N, int k, int pass, int force_last,
                 uint32_t* __restrict__ sc, int* status) {
  __shared__ uint32_t h[256];
  __shared__ uint32_t scan[256];
  __shared__ bool is_last;
  const int tid = threadIdx.x;
  h[tid] = 0;
  // the passes of one selection run as programmatic dependents: the scores were complete before pass 0 started,
  // so they are read before waiting for the previous pass's bucket choice
  dep_launch();
  const int shift = 24 - 8 * pass;
  const uint32_t mask = pass == 0 ? 0u : (0xFFFFFFFFu << (32 - 8 * pass));
  bool nonfinite = false;
  const int base = blockIdx.x * TOPK_CHUNK;
  uint32_t keys[TK_PER_THREAD];
#pragma unroll
  for (int e = 0; e < TK_PER_THREAD; ++e) {
    const int i = base + e * TK_THREADS + tid;
    keys[e] = i < N ? load_key(scores, i, N, force_last != 0, &nonfinite) : 0u;
  }
  dep_wait();
  __syncthreads();
  const uint32_t prefix = pass == 0 ? 0u : __ldcg(&sc[SC_PREFIX]);   // L2: this SM's L1 may hold the older value
#pragma unroll
  for (int e = 0; e < TK_PER_THREAD; ++e) {
    const int i = base + e * TK_THREADS + tid;
    if (i < N && (keys[e] & mask) == prefix) atomicAdd(&h[(keys[e] >> shift) & 0xFFu], 1u);
  }
  if (nonfinite && pass == 0) set_status(status, SPTS_ERR_NONFINITE);
  __syncthreads();
  if (h[tid] != 0) atomicAdd(&sc[SC_HIST + pass * 256 + tid], h[tid]);
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    uint32_t done = atomicAdd(&sc[SC_DONE], 1u);
    is_last = (done == gridDim.x - 1);
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  // inclusive scan from the top digit downwards: scan[t] = sum of hist[255 - t .. 255]
  uint32_t mine = ((volatile uint32_t*)sc)[SC_HIST + pass * 256 + (255 - tid)];
  scan[tid] = mine;
  __syncthreads();
  for (int o = 1; o < 256; o <<= 1) {
    uint32_t v = tid >= o ? scan[tid - o] : 0u;
    __syncthreads();
    scan[tid] += v;
    __syncthreads();
  }
  const uint32_t krem = pass == 0 ? (uint32_t)k : ((volatile uint32_t*)sc)[SC_KREM];
  const uint32_t above = scan[tid] - mine;  // keys in strictly higher buckets
  __syncthreads();
  if (above < krem && krem <= scan[tid]) {  // exactly one thread
    sc[SC_PREFIX] = prefix | ((uint32_t)(255 - tid) << shift);
    sc[SC_KREM] = krem - above;
  }
  if (tid == 0) sc[SC_DONE] = 0u;
}

// Per-chunk counts of keys above / equal to the threshold; the last block turns them into
// output offsets so that the emit kernel writes ascending indices without further sync.
__global__ void __launch_bounds__(TK_THREADS)
topk_count_kernel(const float* __restrict__ scores, int N, int force_last, uint32_t* __restrict__ sc) {
  __shared__ uint32_t s_gt[TK_THREADS / 32], s_eq[TK_THREADS / 32];
  __shared__ bool is_last;
  __shared__ uint32_t carry_out, carry_eq;
  __shared__ uint32_t sa[TK_THREADS], sb[TK_THREADS];
  const int tid = threadIdx.x;
  uint32_t* cta_a = sc + SC_CTA;
  uint32_t* cta_b = sc + SC_CTA + TOPK_MAX_CTAS;
  bool nf = false;
  const int base = blockIdx.x * TOPK_CHUNK;
  dep_launch();
  uint32_t keys[TK_PER_THREAD];
#pragma unroll
  for (int e = 0; e < TK_PER_THREAD; ++e) {
    const int i = base + e * TK_THREADS + tid;
    keys[e] = i < N ? load_key(scores, i, N, force_last != 0, &nf) : 0u;
  }
  dep_wait();                                  // the threshold comes from the last histogram pass
  const uint32_t T = __ldcg(&sc[SC_PREFIX]);   // (read at L2: an L1 line may predate the previous kernel's write)
  uint32_t gt = 0, eq = 0;
#pragma unroll
  for (int e = 0; e < TK_PER_THREAD; ++e) {
    const int i = base + e * TK_THREADS + tid;
    if (i < N) {
      gt += keys[e] > T;
      eq += keys[e] == T;
    }
  }
  gt = __reduce_add_sync(0xffffffffu, gt);
  eq = __reduce_add_sync(0xffffffffu, eq);
  if ((tid & 31) == 0) { s_gt[tid >> 5] = gt; s_eq[tid >> 5] = eq; }
  __syncthreads();
  if (tid == 0) {
    uint32_t a = 0, b = 0;
    for (int w = 0; w < TK_THREADS / 32; ++w) { a += s_gt[w]; b += s_eq[w]; }
    cta_a[blockIdx.x] = a;
    cta_b[blockIdx.x] = b;
    __threadfence();
    uint32_t done = atomicAdd(&sc[SC_DONE], 1u);
    is_last = (done == gridDim.x - 1);
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const uint32_t need_eq = ((volatile uint32_t*)sc)[SC_KREM];
  if (tid == 0) { carry_out = 0; carry_eq = 0; }
  __syncthreads();
  const int nb = gridDim.x;
  for (int c0 = 0; c0 < nb; c0 += TK_THREADS) {
    int b = c0 + tid;
    uint32_t g = 0, e = 0;
    if (b < nb) { g = ((volatile uint32_t*)cta_a)[b]; e = ((volatile uint32_t*)cta_b)[b]; }
    // exclusive scan of eq counts first (needed to clip the equal keys taken per chunk)
    sb[tid] = e;
    __syncthreads();
    for (int o = 1; o < TK_THREADS; o <<= 1) {
      uint32_t v = tid >= o ? sb[tid - o] : 0u;
      __syncthreads();
      sb[tid] += v;
      __syncthreads();
    }
    uint32_t eq_base = carry_eq + sb[tid] - e;
    uint32_t take = 0;
    if (eq_base < need_eq) take = min(e, need_eq - eq_base);
    sa[tid] = g + take;
    __syncthreads();
    for (int o = 1; o < TK_THREADS; o <<= 1) {
      uint32_t v = tid >= o ? sa[tid - o] : 0u;
      __syncthreads();
      sa[tid] += v;
      __syncthreads();
    }
    uint32_t out_base = carry_out + sa[tid] - (g + take);
    if (b < nb) { cta_a[b] = out_base; cta_b[b] = eq_base; }
    __syncthreads();
    if (tid == TK_THREADS - 1) { carry_out += sa[tid]; carry_eq += sb[tid]; }
    __syncthreads();
  }
  if (tid == 0) sc[SC_DONE] = 0u;
}

__global__ void __launch_bounds__(TK_THREADS)
topk_emit_kernel(const float* __restrict__ scores, int N, int k, int force_last,
                 const uint32_t* __restrict__ sc, int32_t* __restrict__ idx_out) {
  __shared__ uint32_t s_sel[TK_THREADS], s_eq[TK_THREADS];
  const int tid = threadIdx.x;
  bool nf = false;
  // thread t owns TK_PER_THREAD consecutive elements so that a scan over threads is index order
  const int i0 = blockIdx.x * TOPK_CHUNK + tid * TK_PER_THREAD;
  dep_launch();
  uint32_t keys[TK_PER_THREAD];
#pragma unroll
  for (int e = 0; e < TK_PER_THREAD; ++e) {
    const int i = i0 + e;
    keys[e] = i < N ? load_key(scores, i, N, force_last != 0, &nf) : 0u;
  }
  dep_wait();                                  // offsets come from the count kernel
  const uint32_t T = __ldcg(&sc[SC_PREFIX]);
  const uint32_t need_eq = __ldcg(&sc[SC_KREM]);
  const uint32_t out_base = __ldcg(&sc[SC_CTA + blockIdx.x]);
  const uint32_t eq_base = __ldcg(&sc[SC_CTA + TOPK_MAX_CTAS + blockIdx.x]);
  uint32_t eq = 0;
#pragma unroll
  for (int e = 0; e < TK_PER_THREAD; ++e) eq += (i0 + e < N && keys[e] == T);
  s_eq[tid] = eq;
  __syncthreads();
  for (int o = 1; o < TK_THREADS; o <<= 1) {
    uint32_t v = tid >= o ? s_eq[tid - o] : 0u;
    __syncthreads();
    s_eq[tid] += v;
    __syncthreads();
  }
  uint32_t eq_rank = eq_base + s_eq[tid] - eq;  // rank of my first equal key among all equal keys
  uint32_t flags = 0, sel = 0;
#pragma unroll
  for (int e = 0; e < TK_PER_THREAD; ++e) {
    int i = i0 + e;
    if (i < N) {
      bool take = keys[e] > T;
      if (keys[e] == T) { take = eq_rank < need_eq; ++eq_rank; }
      if (take) { flags |= 1u << e; ++sel; }
    }
  }
  s_sel[tid] = sel;
  __syncthreads();
  for (int o = 1; o < TK_THREADS; o <<= 1) {
    uint32_t v = tid >= o ? s_sel[tid - o] : 0u;
    __syncthreads();
    s_sel[tid] += v;
    __syncthreads();
  }
  uint32_t w = out_base + s_sel[tid] - sel;
#pragma unroll
  for (int e = 0; e < TK_PER_THREAD; ++e) {
    if (flags & (1u << e)) {
      if (w < (uint32_t)k) idx_out[w] = i0 + e;
      ++w;
    }
  }
}

__global__ void iota_kernel(int32_t* out, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = i;
}

// dst[i, :] = src[idx[i], :], 16 bytes per thread.
__global__ void gather_rows_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ idx,
                                   int n_rows, int row_vec, uint4* __restrict__ dst) {
  size_t total = (size_t)n_rows * row_vec;
  for (size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (size_t)gridDim.x * blockDim.x) {
    int r = (int)(t / row_vec);
    int c = (int)(t - (size_t)r * row_vec);
    dst[t] = src[(size_t)idx[r] * row_vec + c];
  }
}

__global__ void gather_i32_kernel(const int32_t* __restrict__ src, const int32_t* __restrict__ idx,
                                  int n, int32_t* __restrict__ dst) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = src[idx[i]];
}

// ---- one selection per sequence of a packed batch, one CTA each (sequences of up to TOPK_SEG_MAX scores: the keys
// sit in shared memory).  Same rule as the kernels above: 8-bit radix select on the order-preserving keys finds the
// k-th largest key and how many of the keys equal to it are taken (the ones with the lowest indices), then the
// selected indices are written in ascending order -- numbered from the sequence's own first row into out_local
// (optional) and from the batch's first row into out_global (optional), at out_off[b].
constexpr int SEG_THREADS = 512;
__global__ void __launch_bounds__(SEG_THREADS)
topk_segmented_kernel(const float* __restrict__ scores, const int32_t* __restrict__ seq_start,
                      const int32_t* __restrict__ k_arr, const int32_t* __restrict__ out_off, int force_last,
                      int32_t* __restrict__ out_local, int32_t* __restrict__ out_global, int* status) {
  extern __shared__ uint32_t seg_keys[];
  __shared__ uint32_t hist[256];
  __shared__ uint32_t scan[256];
  __shared__ uint32_t s_prefix, s_krem;
  __shared__ uint32_t wsum_gt[SEG_THREADS / 32], wsum_eq[SEG_THREADS / 32];
  __shared__ uint32_t carry_gt, carry_eq;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int b = blockIdx.x;
  const int s0 = seq_start[b];
  const int N = seq_start[b + 1] - s0;
  const int k = k_arr[b];
  const int o0 = out_off[b];
  const float* sc = scores + s0;
  if (k >= N) {                                  // TopK of everything: the identity list
    for (int i = tid; i < N; i += SEG_THREADS) {
      if (out_local) out_local[o0 + i] = i;
      if (out_global) out_global[o0 + i] = s0 + i;
    }
    return;
  }
  bool nonfinite = false;
  for (int i = tid; i < N; i += SEG_THREADS) seg_keys[i] = load_key(sc, i, N, force_last != 0, &nonfinite);
  if (nonfinite) set_status(status, SPTS_ERR_NONFINITE);
  if (tid == 0) { s_prefix = 0u; s_krem = (uint32_t)k; }
  __syncthreads();
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const uint32_t mask = pass == 0 ? 0u : (0xFFFFFFFFu << (32 - 8 * pass));
    if (tid < 256) hist[tid] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    for (int i = tid; i < N; i += SEG_THREADS) {
      const uint32_t key = seg_keys[i];
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 0xFFu], 1u);
    }
    __syncthreads();
    // inclusive scan from the top digit downwards: scan[t] = sum of hist[255 - t .. 255]
    uint32_t mine = 0u;
    if (tid < 256) { mine = hist[255 - tid]; scan[tid] = mine; }
    __syncthreads();
    for (int o = 1; o < 256; o <<= 1) {
      uint32_t v = (tid < 256 && tid >= o) ? scan[tid - o] : 0u;
      __syncthreads();
      if (tid < 256) scan[tid] += v;
      __syncthreads();
    }
    const uint32_t krem = s_krem;
    __syncthreads();
    if (tid < 256) {
      const uint32_t above = scan[tid] - mine;    // keys in strictly higher buckets
      if (above < krem && krem <= scan[tid]) {    // exactly one thread
        s_prefix = prefix | ((uint32_t)(255 - tid) << shift);
        s_krem = krem - above;
      }
    }
    __syncthreads();
  }
  const uint32_t thr = s_prefix, take_eq = s_krem;
  if (tid == 0) { carry_gt = 0u; carry_eq = 0u; }
  __syncthreads();
  // ascending emit: element i goes to (keys above the threshold before it) + (taken equals before it)
  for (int base = 0; base < N; base += SEG_THREADS) {
    const int i = base + tid;
    const uint32_t key = i < N ? seg_keys[i] : 0u;
    const bool gt = i < N && key > thr, eq = i < N && key == thr;
    const uint32_t bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
    if (lane == 0) { wsum_gt[wid] = __popc(bg); wsum_eq[wid] = __popc(be); }
    __syncthreads();
    uint32_t pre_gt = carry_gt, pre_eq = carry_eq;
    for (int w = 0; w < wid; ++w) { pre_gt += wsum_gt[w]; pre_eq += wsum_eq[w]; }
    const uint32_t lt = (1u << lane) - 1u;
    pre_gt += __popc(bg & lt);
    pre_eq += __popc(be & lt);
    if (gt || (eq && pre_eq < take_eq)) {
      const uint32_t pos = pre_gt + (pre_eq < take_eq ? pre_eq : take_eq);
      if (out_local) out_local[o0 + pos] = i;
      if (out_global) out_global[o0 + pos] = s0 + i;
    }
    __syncthreads();
    if (tid == 0) {
      uint32_t g = 0u, e = 0u;
      for (int w = 0; w < SEG_THREADS / 32; ++w) { g += wsum_gt[w]; e += wsum_eq[w]; }
      carry_gt += g;
      carry_eq += e;
    }
    __syncthreads();
  }
}

}  // namespace

spts_status launch_topk_segmented(spts_ctx* ctx, const float* scores, const int32_t* seq_start, const int32_t* k_arr,
                                  const int32_t* out_off, int n_seq, int max_len, uint32_t flags, int32_t* out_local,
                                  int32_t* out_global) {
  if (n_seq <= 0) return SPTS_OK;
  if (max_len > TOPK_SEG_MAX) return SPTS_ERR_SHAPE;
  const size_t smem = (size_t)max_len * sizeof(uint32_t);
  topk_segmented_kernel<<<n_seq, SEG_THREADS, smem, ctx->stream>>>(scores, seq_start, k_arr, out_off,
                                                                  (flags & SPTS_FORCE_LAST) ? 1 : 0, out_local, out_global,
                                                                  ctx->ws.status);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_topk(spts_ctx* ctx, const float* scores, int N, int k, uint32_t flags,
                        int32_t* idx_out, uint32_t* scratch) {
  if (scores == nullptr || idx_out == nullptr || N < 1 || k < 1 || k > N) return SPTS_ERR_INVALID_ARG;
  const int nb = ceil_div(N, TOPK_CHUNK);
  if (nb > TOPK_MAX_CTAS) return SPTS_ERR_SHAPE;
  cudaStream_t st = ctx->stream;
  if (k == N) {  // TopK of everything: the identity list
    iota_kernel<<<ceil_div(N, 256), 256, 0, st>>>(idx_out, N);
    SPTS_CUDA_OK(ctx);
    return SPTS_OK;
  }
  const int fl = (flags & SPTS_FORCE_LAST) ? 1 : 0;
  if (cudaMemsetAsync(scratch, 0, (4 * 256 + 16) * sizeof(uint32_t), st) != cudaSuccess) return SPTS_ERR_CUDA;
  topk_hist_kernel<<<nb, TK_THREADS, 0, st>>>(scores, N, k, 0, fl, scratch, ctx->ws.status);   // after the memset
  SPTS_CUDA_OK(ctx);
  for (int pass = 1; pass < 4; ++pass) {
    if (launch_dependent(topk_hist_kernel, dim3(nb), dim3(TK_THREADS), st, scores, N, k, pass, fl, scratch,
                         ctx->ws.status) != cudaSuccess)
      return SPTS_ERR_CUDA;
    ctx->launches++;
  }
  if (launch_dependent(topk_count_kernel, dim3(nb), dim3(TK_THREADS), st, scores, N, fl, scratch) != cudaSuccess)
    return SPTS_ERR_CUDA;
  ctx->launches++;
  if (launch_dependent(topk_emit_kernel, dim3(nb), dim3(TK_THREADS), st, scores, N, k, fl, (const uint32_t*)scratch,
                       idx_out) != cudaSuccess)
    return SPTS_ERR_CUDA;
  ctx->launches++;
  return SPTS_OK;
}

spts_status launch_gather_rows(spts_ctx* ctx, const void* src, const int32_t* idx, int n_rows,
                               int row_bytes, void* dst) {
  if (row_bytes % 16 != 0) return SPTS_ERR_SHAPE;
  if (n_rows == 0) return SPTS_OK;
  int row_vec = row_bytes / 16;
  size_t total = (size_t)n_rows * row_vec;
  int blocks = (int)((total + 255) / 256);
  int cap = ctx->sm_count * 16;
  if (blocks > cap) blocks = cap;
  gather_rows_kernel<<<blocks, 256, 0, ctx->stream>>>((const uint4*)src, idx, n_rows, row_vec, (uint4*)dst);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

// dst[i] = src[i] + offset: a sequence's own row numbers -> rows of the packed batch
__global__ void offset_i32_kernel(const int32_t* __restrict__ src, int n, int offset, int32_t* __restrict__ dst) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = src[i] + offset;
}

spts_status launch_offset_i32(spts_ctx* ctx, const int32_t* src, int n, int offset, int32_t* dst) {
  if (n == 0) return SPTS_OK;
  offset_i32_kernel<<<ceil_div(n, 256), 256, 0, ctx->stream>>>(src, n, offset, dst);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

// SPTS_DEBUG_CHECKS: an index list must lie in [0, N) and ascend strictly; a violation is recorded, never trapped on
__global__ void check_index_list_kernel(const int32_t* __restrict__ idx, int n, int N, int* status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int v = idx[i];
  bool bad = v < 0 || v >= N;
  if (i > 0 && idx[i - 1] >= v) bad = true;
  if (bad) set_status(status, SPTS_ERR_INDEX);
}

spts_status launch_check_index_list(spts_ctx* ctx, const int32_t* idx, int n, int N) {
  if (n == 0) return SPTS_OK;
  check_index_list_kernel<<<ceil_div(n, 256), 256, 0, ctx->stream>>>(idx, n, N, ctx->ws.status);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_gather_i32(spts_ctx* ctx, const int32_t* src, const int32_t* idx, int n, int32_t* dst) {
  if (n == 0) return SPTS_OK;
  gather_i32_kernel<<<ceil_div(n, 256), 256, 0, ctx->stream>>>(src, idx, n, dst);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

}  // namespace spts

// ---------------------------------------------------------------------------------------------
// Allocation-free top-k (declared in spts.h as spts_topk_select_static)
//
// Every other call of the library works out of a workspace the caller allocated.  Some hosts cannot
// allocate at all: an inference server whose device memory was planned and frozen at start-up, a
// plugin that only ever receives input and output buffers from its framework, a real-time loop that
// must not touch the allocator.  For them the radix-select scratch lives in this file-scope device
// array, which every GPU that loads the library holds from load to exit.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) uint32_t spts_static_topk_scratch[spts::TOPK_SCRATCH_WORDS];
static_assert(sizeof(uint32_t) * spts::TOPK_SCRATCH_WORDS == SPTS_TOPK_STATIC_SCRATCH_BYTES, "scratch size as documented");
static_assert((long)spts::TOPK_MAX_CTAS * spts::TOPK_CHUNK == SPTS_TOPK_STATIC_MAX_N, "size limit as documented");

namespace spts {
namespace {

constexpr int STATIC_MAX_DEVICES = 64;
std::mutex g_static_mu;
uint32_t* g_static_ptr[STATIC_MAX_DEVICES];   // device address of the array, per device ordinal

// In host code the array's name is only a handle for the runtime, not a device address: the
// address each device gave it is looked up once per device, with that device current.
spts_status static_scratch_address(uint32_t** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) return SPTS_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (g_static_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, spts_static_topk_scratch) != cudaSuccess || p == nullptr) return SPTS_ERR_CUDA;
    g_static_ptr[dev] = static_cast<uint32_t*>(p);
  }
  *out = g_static_ptr[dev];
  return SPTS_OK;
}

}  // namespace
}  // namespace spts

extern "C" spts_status spts_topk_select_static(const float* scores, int N, int k, uint32_t flags, int32_t* idx_out,
                                               void* cuda_stream) {
  using namespace spts;
  if (scores == nullptr || idx_out == nullptr || N < 1 || k < 1 || k > N) return SPTS_ERR_INVALID_ARG;
  if (N > SPTS_TOPK_STATIC_MAX_N) return SPTS_ERR_SHAPE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (k == N) {   // the identity list needs no scratch
    iota_kernel<<<ceil_div(N, 256), 256, 0, st>>>(idx_out, N);
    return cudaGetLastError() == cudaSuccess ? SPTS_OK : SPTS_ERR_CUDA;
  }
  uint32_t* scratch = nullptr;
  spts_status s = static_scratch_address(&scratch);
  if (s != SPTS_OK) return s;
  const int nb = ceil_div(N, TOPK_CHUNK);
  const int fl = (flags & SPTS_FORCE_LAST) ? 1 : 0;
  // the array keeps the previous call's contents: histograms, prefix and counters must start at zero
  if (cudaMemsetAsync(scratch, 0, (4 * 256 + 16) * sizeof(uint32_t), st) != cudaSuccess) return SPTS_ERR_CUDA;
  for (int pass = 0; pass < 4; ++pass)
    topk_hist_kernel<<<nb, TK_THREADS, 0, st>>>(scores, N, k, pass, fl, scratch, nullptr);
  topk_count_kernel<<<nb, TK_THREADS, 0, st>>>(scores, N, fl, scratch);
  topk_emit_kernel<<<nb, TK_THREADS, 0, st>>>(scores, N, k, fl, scratch, idx_out);
  return cudaGetLastError() == cudaSuccess ? SPTS_OK : SPTS_ERR_CUDA;
}
