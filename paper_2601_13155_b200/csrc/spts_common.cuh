// Shared declarations of the SPTS CUDA library (internal; the public boundary is include/spts.h).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include <vector>

#include "spts.h"

namespace spts {

typedef __nv_bfloat16 bf16;

// ---------------------------------------------------------------------------------------------
// device status word: kernels record problems here instead of trapping
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void set_status(int* status, int code) {
  if (status != nullptr) atomicCAS(status, 0, code);
}

// ---------------------------------------------------------------------------------------------
// storage-type helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__host__ __device__ __forceinline__ size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
__host__ __device__ __forceinline__ int ceil_div(int a, int b) { return (a + b - 1) / b; }

// ---------------------------------------------------------------------------------------------
// context
// ---------------------------------------------------------------------------------------------
struct Workspace {
  // all device pointers, carved from the caller's workspace
  int* status;          // [1] device status word
  float* rstd;          // [Nmax]
  float* q;             // [H*d]
  float2* rope_cs;      // [Nmax, d/2] cos/sin of the rotary angles
  void* vgu_pad;        // [2, Dlow, 2r] zero-padded proxy factors (gate | up)
  float* pw_logits;     // [PAP_MAX_WINDOW * G, Nmax] probe logits of one KV head's window queries
  float* pw_stats;      // [2 * PAP_MAX_WINDOW * G]
  void* q_win;          // [PAP_MAX_WINDOW, H*d] window queries after RoPE
  void* q_kv;           // the same regrouped by KV head
  int32_t* idx_w;       // [PAP_MAX_WINDOW] the window's candidate indices
  void* ugu;            // [2r, D] the proxy's first factors stacked (Ug^T over Uu^T): one GEMM reads x once
  void* g2;             // [2r, r] Gram matrix Ud^T Ud, high part over low part (tensor-core mode)
  float* logits;        // [H, Nmax]
  float* head_stats;    // [2*H] max and sum of exp per head
  float* s_mha;         // [Nmax]
  float* s_ffn;         // [Nmax]
  float* csq;           // [Nmax * csq_parts] partial sums of squares of the proxy output
  int32_t* idx_a;       // [Nmax]
  int32_t* idx_f;       // [Nmax]
  int32_t* idx_p;       // [Nmax]
  uint32_t* topk_scratch;  // radix-select scratch
  void* k_all;          // [Nmax, Hkv*d]
  void* q_act;          // [Nmax, H*d]
  void* v_t;            // [Hkv*d, Nmax_pad] transposed V for the tensor-core attention
  void* o_att;          // [Nmax, H*d]
  void* hm;             // [Nmax, Dff]
  void* t1;             // [Nmax, 2r]
  void* hlow;           // [Nmax, Dlow]
  void* t2;             // [Nmax, r]
  float* acc32;         // fp32 accumulator scratch of the reference GEMM path
  size_t acc32_elems;
  void* dec;            // decode-step scratch
  float* logits_v;      // [vocab]
  void* xrow;           // [D] one hidden row in the storage type
  int csq_parts;
  // packed batches: host tables copied in per call, row -> sequence map, V^T column of every active row
  int32_t* batch_i32;   // [6 * (BATCH_MAX_SEQ + 1)]
  void** batch_ptr;     // [3 * BATCH_MAX_SEQ] cache pointers (k, v, pos)
  int32_t* row_seq;     // [Nmax]
  int32_t* vt_col;      // [Nmax]
  int vt_ld_max;        // columns of v_t
  int4* attn_tiles;     // [Nmax / 128 + BATCH_MAX_SEQ] query tiles of a packed batch's attention launch
};

}  // namespace spts

struct spts_ctx {
  spts_model_desc desc;
  int max_seq;
  cudaStream_t stream;
  spts::Workspace ws;
  bool reference_kernels;   // plain CUDA-core kernels (always true in fp32 mode)
  bool ffn_score_pap_only;   // T_f from S_mha alone (no proxy FFN)
  bool debug_checks;        // every selected index list is checked on the device (SPTS_ERR_INDEX in the status word)
  char* ws_base;            // the caller's workspace and the byte offsets of the guard bands that follow its slices
  std::vector<size_t> guard_offsets;
  // set by spts_prefill between two layers: ws.rstd is current for the rows of rstd_x [rstd_n] except the listed ones
  const int32_t* rstd_rows; int rstd_nrows; const void* rstd_x; int rstd_n;
  // rotary table reuse inside spts_prefill: positions only change at a stage end, so the table computed for
  // (pos pointer, N) stays valid for the following layers of the stage
  bool rope_trust;
  const int32_t* rope_pos;
  int rope_n;
  int pap_window;           // number of trailing queries the probe averages over (1 = the paper's default)
  int64_t launches;
  int sm_count;
  void* encode_tiled;       // cuTensorMapEncodeTiled entry point (tensor-core mode)
  void* prof;               // per-operation CUDA-event timing (host state)
};

namespace spts {

static const int BATCH_MAX_SEQ = 1024;        // sequences per packed batch that take the one-launch-per-step route
static const int PAP_MAX_WINDOW = 64;         // largest query window of the probe (the paper ablates 1, 4 and 64)

// top-k scratch size in uint32 words
static const int TOPK_CHUNK = 2048;           // elements per CTA in the select / emit kernels
static const int TOPK_MAX_CTAS = 4096;        // supports N up to 8M
static const int TOPK_SCRATCH_WORDS = 4 * 256 + 16 + 2 * TOPK_MAX_CTAS;

// ---- kernels_select.cu
spts_status launch_topk(spts_ctx* ctx, const float* scores, int N, int k, uint32_t flags,
                        int32_t* idx_out, uint32_t* scratch);
spts_status launch_gather_rows(spts_ctx* ctx, const void* src, const int32_t* idx, int n_rows,
                               int row_bytes, void* dst);
spts_status launch_gather_i32(spts_ctx* ctx, const int32_t* src, const int32_t* idx, int n, int32_t* dst);
spts_status launch_offset_i32(spts_ctx* ctx, const int32_t* src, int n, int offset, int32_t* dst);
static const int TOPK_SEG_MAX = 8192;         // longest sequence the one-CTA-per-sequence selection takes
spts_status launch_topk_segmented(spts_ctx* ctx, const float* scores, const int32_t* seq_start, const int32_t* k_arr,
                                  const int32_t* out_off, int n_seq, int max_len, uint32_t flags, int32_t* out_local,
                                  int32_t* out_global);
spts_status launch_check_index_list(spts_ctx* ctx, const int32_t* idx, int n, int N);   // debug option only
spts_status launch_wait_selftest(spts_ctx* ctx, uint32_t limit_us);

static const int GUARD_BYTES = 256;           // band after every workspace slice
static const int GUARD_PATTERN = 0xA5;

// ---- kernels_probe.cu
spts_status launch_rstd(spts_ctx* ctx, const void* X, int N, float* rstd);
spts_status launch_rstd_rows(spts_ctx* ctx, const void* X, const int32_t* idx, int n, float* rstd);
spts_status launch_rope_table(spts_ctx* ctx, const int32_t* pos, int N, float2* cs);
spts_status launch_q_last(spts_ctx* ctx, const void* X, const float2* cs, int N, const void* wq,
                          const float* rstd, float* q);
spts_status launch_pad_proxy(spts_ctx* ctx, const void* vg, const void* vu, void* out);
spts_status launch_gram(spts_ctx* ctx, const void* ud, void* g2);   // g2 [2r, r]: bf16(G) over bf16(G - bf16(G)), G = Ud^T Ud
spts_status launch_pap_softmax(spts_ctx* ctx, const float* logits, int ld_logits, int N, float* S);
spts_status launch_pap_window_softmax(spts_ctx* ctx, const float* logits, int ld_logits, int N, int w, int accumulate,
                                      float* stats, float* S);
spts_status launch_pap_regroup(spts_ctx* ctx, const void* q_win, int w, void* q_kv);
spts_status launch_batch_vt_col(spts_ctx* ctx, const int32_t* act_off, const int32_t* vt0, int n_seq, int n_act, int32_t* vt_col);
spts_status launch_batch_row_seq(spts_ctx* ctx, const int32_t* seq_start, int n_seq, int total, int32_t* row_seq);
spts_status launch_q_last_batch(spts_ctx* ctx, const void* X, const float2* cs, const int32_t* seq_start, int n_seq,
                                const void* wq, const float* rstd, float* q);
spts_status launch_pap_softmax_batch(spts_ctx* ctx, const float* logits, int ld_logits, const int32_t* seq_start,
                                     int n_seq, int total, const int32_t* row_seq, float* stats, float* S);
spts_status launch_batch_cache_fill(spts_ctx* ctx, const void* k_all, const void* v_act, const int32_t* pos,
                                    const int32_t* idx_global, const int32_t* act_off, int n_seq, int n_act,
                                    void* const* k_ptrs, void* const* v_ptrs, int32_t* const* pos_ptrs);
spts_status launch_iota_from(spts_ctx* ctx, int32_t* out, int n, int first);
spts_status launch_transpose_bf16(spts_ctx* ctx, const void* in, int rows, int cols, void* out_t, int ldt);
spts_status launch_ffn_score(spts_ctx* ctx, const float* csq, int parts, const float* S_mha, int N,
                             float* C_out, float* S_ffn);
spts_status launch_fold_gain(spts_ctx* ctx, void* W, const float* g, int out_f, int in_f);
spts_status launch_head(spts_ctx* ctx, const void* x_row, const void* lm_head, float* logits,
                        int32_t* token_out);

// ---- kernels_ref.cu : plain CUDA-core path (fp32 verification mode, bf16 cross-check)
enum RefEpi {
  REF_STORE = 0,       // out[i, j] = T(acc * rowscale)
  REF_ROPE = 1,        // out[i, j] = T(rope(acc * rowscale)) ; optional PAP logits from unrounded values
  REF_SWIGLU = 2,      // out[i, j] = T(silu(acc1 * rowscale) * (acc2 * rowscale))
  REF_RESID = 3,       // X[dst(i), j] = T(X[dst(i), j] + acc)
  REF_SUMSQ = 4        // csq[i, part] = sum_j acc^2 (deterministic partials)
};
struct RefGemmArgs {
  const void* A; int lda;            // A [*, K] rows addressed through idx (or i when idx == nullptr)
  const int32_t* idx;                // gather list for A rows, row scales and positions
  const int32_t* dst_idx;            // REF_RESID: residual rows to update (nullptr: row i)
  const void* W; const void* W2;     // [Nout, K] row-major; W2 for REF_SWIGLU
  int M, Nout, K;
  const float* rowscale;             // [*] indexed like A rows, or nullptr
  void* out; int ldo;                // output matrix (REF_RESID: the residual stream X, row stride ldo)
  void* out_t; int ldt;              // optional transposed copy out_t[j, i] (REF_STORE)
  int head_dim;                      // REF_ROPE: rotary table rows are indexed like A rows
  const float* q; float* logits; int ld_logits; int group;   // REF_ROPE + PAP: q [H, d], logits [H, ld]
  float* csq; int csq_parts;         // REF_SUMSQ
  float* sal_t; int ld_sal;          // REF_SWIGLU: write |silu(g) u| as fp32 [column, row] instead of `out`
  int ldw;                           // row stride of W in elements (0: K)
  float* out_f32;                    // REF_STORE: write fp32 [M, ldo] instead of `out`
};
spts_status launch_ref_gemm(spts_ctx* ctx, int epi, const RefGemmArgs& a);
spts_status launch_ref_attention(spts_ctx* ctx, const void* Q, const void* K, const void* V, int m,
                                 void* O);

// ---- kernels_decode.cu
constexpr int ARGMAX_BLOCKS = 128;     // partial results of the two-step argmax over the logits
size_t decode_scratch_floats(const spts_model_desc& d);
float* argmax_scratch(spts_ctx* ctx);
spts_status launch_decode_load(spts_ctx* ctx, const void* x);     // x [D] -> fp32 residual scratch
spts_status launch_decode_store(spts_ctx* ctx, void* x);          // fp32 residual scratch -> x [D]
spts_status launch_decode_layer(spts_ctx* ctx, const spts_layer_weights* w, spts_kv_layer* cache,
                                int32_t pos);
spts_status launch_head_logits(spts_ctx* ctx, const float* x32, const void* lm_head, float* logits);

// ---- kernels_proxy.cu : offline proxy-FFN construction
spts_status launch_proxy_importance(spts_ctx* ctx, const float* zt, int ld, int n_cal, int k, int n_channels,
                                    float* importance);
spts_status launch_proxy_factor(spts_ctx* ctx, const void* W, const int32_t* channels, int down, int sweeps,
                                float* A, float* V, float* sigma, int32_t* order, unsigned int* offdiag, int r,
                                void* u_out, void* v_out, float* sigma_sorted);

// ---- kernels_tc_gemm.cu / kernels_tc_attn.cu : tcgen05 path (bf16)
enum TcEpi { TC_STORE = 0, TC_ROPE = 1, TC_SWIGLU = 2, TC_RESID = 3, TC_SUMSQ = 4, TC_QFORM = 5 };
struct TcGemmArgs {
  const bf16* A; int lda; int a_rows;   // A [a_rows, K]
  const int32_t* idx;                   // optional gather list of A rows
  const int32_t* dst_idx;               // TC_RESID scatter rows
  const bf16* W; const bf16* W2;        // [Nout, K]
  int M, Nout, K;
  const float* rowscale;
  bf16* out; int ldo;
  bf16* out_t; int ldt;
  const float* q; float* logits; int ld_logits; int group;
  float* csq; int csq_parts;
  float* sal_t; int ld_sal;             // TC_SWIGLU: saliency output (proxy construction)
  int ldw;                              // row stride of W in elements (0: K)
  float* out_f32;                       // TC_STORE: fp32 output [M, ldo] instead of `out`
  const int32_t* row_seq; int q_stride; // TC_ROPE + PAP over a packed batch: row -> sequence, stride between the q's
  const int32_t* out_t_col;             // TC_STORE: column of out_t per row (nullptr: the row number)
};
spts_status launch_tc_gemm(spts_ctx* ctx, int epi, const TcGemmArgs& a);
spts_status launch_tc_attention(spts_ctx* ctx, const bf16* Q, const bf16* K, const bf16* V, const bf16* Vt, int ldvt,
                                int m, bf16* O);
spts_status launch_tc_attention_packed(spts_ctx* ctx, const bf16* Q, const bf16* K, const bf16* Vt, int ldvt, int n_act,
                                       int vt_cols, const int4* tiles, int n_tiles, bf16* O);
spts_status tc_init(spts_ctx* ctx);          // resolves the tensor-map encoder, sets kernel attributes
int tc_sumsq_parts(int n_out);               // partial sums per row written by TC_SUMSQ

// Programmatic dependent launch for chains of short kernels (the decode step, the passes of a top-k): a kernel
// lets its successor start early (dep_launch), does whatever does not depend on its predecessor (prefetching
// weights, loading keys) and only then waits for the predecessor's results (dep_wait = predecessor complete,
// its writes visible; a no-op in a kernel that was launched the ordinary way).
__device__ __forceinline__ void dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

#define SPTS_CUDA_OK(ctx)                                   \
  do {                                                      \
    cudaError_t e__ = cudaGetLastError();                   \
    if (e__ != cudaSuccess) return SPTS_ERR_CUDA;           \
    (ctx)->launches++;                                      \
  } while (0)

}  // namespace spts
