/*
 * spts.h -- C boundary of the SPTS (Self-Predictive Token Skipping) prefill library for
 * NVIDIA B200 (sm_100a).
 *
 * The library runs the token-selective transformer prefill layer of the SPTS paper:
 * Partial Attention Probing (Section 3.2, Eq. 4-5), Low-rank Transformation Probing
 * (Section 3.3, Eq. 12-15), top-k selection, the reduced attention / FFN blocks with
 * residual scatter (Eq. 2, Algorithm 1), Multi-Stage Delayed Pruning (Section 3.4, Eq. 16)
 * and the decode step over the per-layer compressed KV cache.
 *
 * General rules
 *   - Every pointer named in a signature is a DEVICE pointer unless the comment says "host".
 *     Structs (model_desc, layer_weights, kv_layer, layer_plan) live in HOST memory and hold
 *     device pointers.
 *   - The caller owns every buffer, including the workspace given to spts_create().  The
 *     library allocates no device memory and frees nothing.
 *   - All work is enqueued on the context's CUDA stream and returns without synchronising.
 *     Sizes (N, k, m_attn, m_ffn, n_next) are host integers: Algorithm 1 fixes them from the
 *     schedule (M^l = min(|T^l|, M_fixed), Section 3.4), so no call reads a count back.
 *   - Storage type: dtype SPTS_BF16 (bf16 in HBM, fp32 accumulation, tensor-core kernels) or
 *     SPTS_FP32 (verification mode: fp32 storage and CUDA-core fp32 arithmetic).  Scores,
 *     softmax statistics and norms are fp32 in both modes.
 *   - Weight matrices are row-major [out_features, in_features].  RMSNorm gains are expected
 *     to be folded into the columns of the matrices that consume the normalised rows
 *     (spts_fold_norm_gain()); with unit gains nothing needs to be done.
 *   - Index lists are int32, strictly ascending.  Ties in a top-k go to the lower index.
 *   - Errors detectable on the host (null pointer, k > N, unsupported shape, workspace too
 *     small, misalignment) are returned before anything is launched.  Device-side problems
 *     (a bounded wait that expired, a non-finite score) set a status word that
 *     spts_last_device_status() returns after synchronising the stream; kernels never trap.
 *   - Pointers must be 16-byte aligned; rows of X, K, V are contiguous.
 *   - A context is bound to one device and one stream and is not thread-safe: calls on one context must
 *     not overlap on the host.  Contexts on different streams are independent (each has its workspace).
 *     spts_layer_prefill_skip() and spts_prefill() use the context's workspace for every intermediate
 *     (K of all candidates, the selected rows' Q, the attention output, the SwiGLU intermediate, scores,
 *     index lists), so the workspace grows with max_seq: about 24 KiB per candidate at the 8B shape plus 0.5 GB (of
 *     which 0.47 GB is the SwiGLU intermediate of one 16384-row chunk): 1.30 GB at 32768 candidates, 3.68 GB at 131072.
 */
#ifndef SPTS_H_
#define SPTS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SPTS_OK = 0,
  SPTS_ERR_INVALID_ARG = 1,
  SPTS_ERR_SHAPE = 2,
  SPTS_ERR_WORKSPACE = 3,
  SPTS_ERR_CUDA = 4,
  SPTS_ERR_TIMEOUT = 5,
  SPTS_ERR_NONFINITE = 6,
  SPTS_ERR_UNSUPPORTED = 7,
  SPTS_ERR_INDEX = 8      /* SPTS_DEBUG_CHECKS: an index list was out of range or not strictly ascending */
} spts_status;

enum { SPTS_BF16 = 0, SPTS_FP32 = 1 };

/* flags */
enum {
  SPTS_FORCE_LAST = 1u,   /* the last candidate is always selected (it carries the output state) */
  SPTS_REFERENCE_KERNELS = 2u, /* spts_set_option: run the plain CUDA-core kernels also in bf16 mode */
  SPTS_PAP_WINDOW = 8u,        /* spts_set_option: value = number of trailing queries the probe score averages over
                                  (1..64; 1 = last token only, Eq. 4; larger windows are the query-length ablation of
                                  Appendix C: every query attends causally, K and the queries are taken as stored) */
  SPTS_DEBUG_CHECKS = 32u,     /* spts_set_option: after every selection a small kernel checks the index list
                                  (0 <= idx < N, strictly ascending) and records SPTS_ERR_INDEX in the device status
                                  word; nothing traps.  Off by default (one extra launch per selection) */
  SPTS_FFN_SCORE_PAP_ONLY = 16u /* spts_set_option: T_f = TopK(S_mha, m_ffn) -- the FFN block selects by the attention
                                  probe's score alone (Eq. 4) and the proxy FFN of Eq. 12-14 is not evaluated: the
                                  criterion the paper's proxy-network ablation (Table 4) compares Eq. 14 against */
};

typedef struct {
  int32_t hidden;      /* D */
  int32_t n_q_heads;   /* H */
  int32_t n_kv_heads;  /* Hkv, divides H */
  int32_t head_dim;    /* d */
  int32_t ffn_dim;     /* Dff */
  int32_t ltp_dlow;    /* D_low of the proxy FFN (Eq. 12) */
  int32_t ltp_rank;    /* r of the proxy FFN */
  int32_t n_layers;
  int32_t vocab;
  float rms_eps;
  float rope_theta;
  int32_t dtype;       /* SPTS_BF16 or SPTS_FP32 */
} spts_model_desc;

/* Device pointers, each [out, in] row-major in the model's storage type. */
typedef struct {
  const void* wq;      /* [H*d, D]   */
  const void* wk;      /* [Hkv*d, D] */
  const void* wv;      /* [Hkv*d, D] */
  const void* wo;      /* [D, H*d]   */
  const void* w_gate;  /* [Dff, D]   */
  const void* w_up;    /* [Dff, D]   */
  const void* w_down;  /* [D, Dff]   */
  const void* ug;      /* [r, D]      U_gate^T  */
  const void* vg;      /* [Dlow, r]   V_gate^T  */
  const void* uu;      /* [r, D]      U_up^T    */
  const void* vu;      /* [Dlow, r]   V_up^T    */
  const void* vd;      /* [r, Dlow]   V_down    */
  const void* ud;      /* [D, r]      U_down    */
  const void* prepared; /* optional: the layer's buffer filled by spts_prepare_layer() (NULL: the proxy factors are
                           repacked inside every call that evaluates Eq. 12-14) */
} spts_layer_weights;

/* One layer's KV cache: k, v are [capacity, Hkv, d] in the storage type (K after RoPE),
 * pos [capacity] holds the original position of every cached token.  `len` is host state. */
typedef struct {
  void* k;
  void* v;
  int32_t* pos;
  int32_t len;
  int32_t capacity;
} spts_kv_layer;

/* Per-layer entry of the MSDP schedule (Section 3.4): active budgets already clipped to the
 * candidate count, and the candidate count to prune to after this layer (0 = not a stage end). */
typedef struct {
  int32_t m_attn;
  int32_t m_ffn;
  int32_t prune_to;
} spts_layer_plan;

/* One stage of the MSDP schedule (Section 3.4; the settings of Section 4.1 are given in this form): the last
 * layer of the stage (0-indexed), the fixed active budgets M_fixed of its attention and FFN blocks (<= 0: that
 * block runs on every candidate in this stage) and the candidate count N_{s+1} the stage end prunes to by
 * Eq. 16 (<= 0: the stage end does not prune). */
typedef struct {
  int32_t last_layer;
  int32_t m_attn_fixed;
  int32_t m_ffn_fixed;
  int32_t n_next;
} spts_msdp_stage;

typedef struct {
  const spts_layer_weights* layers; /* host array [n_layers] */
  const void* lm_head;              /* [vocab, D] */
  const void* embed;                /* [vocab, D], used by spts_decode_step */
} spts_model_weights;

/* Operation tags of the per-operation timer (spts_profile_begin / spts_profile_end). */
enum {
  SPTS_OP_PREP = 1,        /* row RMS statistics, rotary table, last-token query            */
  SPTS_OP_KPROJ = 2,       /* K projection of all candidates + RoPE + PAP logits (Eq. 4)   */
  SPTS_OP_PAP_SOFTMAX = 3, /* head-mean softmax of Eq. 4                                    */
  SPTS_OP_TOPK = 4,        /* Eq. 5 / 15 / 16                                               */
  SPTS_OP_KV_GATHER = 5,   /* K^ = K[T_a], cache positions                                  */
  SPTS_OP_QVPROJ = 6,      /* gathered Q (RoPE) and V projections                           */
  SPTS_OP_ATTN = 7,        /* causal GQA attention among the active rows                    */
  SPTS_OP_OPROJ = 8,       /* O projection + residual scatter                               */
  SPTS_OP_LTP = 9,         /* proxy FFN chain, row norms and score fusion (Eq. 12-14)       */
  SPTS_OP_GATEUP = 10,     /* gathered gate/up GEMM + SwiGLU                                */
  SPTS_OP_DOWN = 11,       /* down GEMM + residual scatter                                  */
  SPTS_OP_COMPACT = 12,    /* stage-end row compaction (Eq. 16)                             */
  SPTS_OP_HEAD = 13,       /* final norm, LM head, argmax                                   */
  SPTS_OP_DECODE = 14,     /* all layers of one decode step                                 */
  SPTS_OP_COUNT = 16
};

typedef struct spts_ctx spts_ctx;

/* Bytes of device workspace spts_create() needs for sequences of up to max_seq candidates. */
size_t spts_workspace_bytes(const spts_model_desc* desc, int max_seq);

/* Creates a context.  `workspace` is caller-owned device memory of at least
 * spts_workspace_bytes() bytes, 256-byte aligned; `cuda_stream` is a cudaStream_t (may be 0).
 * Must be called with the target device current.  Returns SPTS_ERR_SHAPE for shapes the
 * kernels do not cover (head_dim must be 64 or 128, H a multiple of Hkv, dimensions
 * multiples of 8; bf16 tensor-core mode additionally needs head_dim 128 and hidden, ffn_dim,
 * ltp_dlow multiples of 64, ltp_rank a multiple of 16). */
spts_status spts_create(const spts_model_desc* desc, int max_seq, void* workspace,
                        size_t workspace_bytes, void* cuda_stream, spts_ctx** out);
void spts_destroy(spts_ctx* ctx);

/* Sets SPTS_REFERENCE_KERNELS, SPTS_FFN_SCORE_PAP_ONLY or SPTS_DEBUG_CHECKS on/off
 * (value 0/1), or SPTS_PAP_WINDOW (value 1..64). */
spts_status spts_set_option(spts_ctx* ctx, uint32_t option, int value);

/* Synchronises the context's stream and returns the device status word (then clears it). */
spts_status spts_last_device_status(spts_ctx* ctx);

/* Guard bands (the paper has no counterpart: a stand-in for a memory checker).  Every slice the library carves out
 * of the caller's workspace is followed by a 256-byte band that spts_create() fills with a fixed pattern and no
 * kernel has any business writing.  spts_check_guards synchronises the stream, reads the bands back and stores the
 * number of bands that no longer hold the pattern in *n_corrupt (HOST memory); a non-zero count means some kernel
 * wrote past the end of its slice. */
spts_status spts_check_guards(spts_ctx* ctx, int32_t* n_corrupt);

/* The check SPTS_DEBUG_CHECKS runs after every selection, on a list the caller provides: idx [n] (device) must lie
 * in [0, N) and ascend strictly, otherwise SPTS_ERR_INDEX is recorded in the device status word (read it with
 * spts_last_device_status).  The kernel only reads the n entries; it never dereferences them. */
spts_status spts_debug_check_index_list(spts_ctx* ctx, const int32_t* idx, int n, int N);

/* Exercises the give-up path of the bounded waits (again no counterpart in the paper).  Every mbarrier wait of the
 * tensor-core kernels ends after a time limit: the waiting thread raises a CTA-wide flag, the other roles see it
 * and return from their own waits, the CTA lets copies in flight land, records SPTS_ERR_TIMEOUT in the device
 * status word and exits normally.  This call launches one tiny CTA that runs exactly that code on two barriers
 * nobody ever arrives on, with the limit shortened to limit_us microseconds (1..100000), so a test can see the
 * status come back and the context stay usable.  The production kernels are not involved. */
spts_status spts_selftest_wait_timeout(spts_ctx* ctx, uint32_t limit_us);

/* Number of kernels the library has launched on this context so far. */
int64_t spts_launch_count(const spts_ctx* ctx);

/* Per-operation timing with CUDA events recorded on the context's stream (the paper has no
 * counterpart; this is measurement plumbing).  spts_profile_begin starts recording event pairs
 * around every operation with tag `op` (-1: every tagged operation); spts_profile_end stops,
 * synchronises the stream and fills four host arrays of SPTS_OP_COUNT entries indexed by tag:
 * elapsed milliseconds, number of timed operations, algorithmic FLOPs and algorithmic bytes. */
spts_status spts_profile_begin(spts_ctx* ctx, int op);
spts_status spts_profile_end(spts_ctx* ctx, float* ms, int64_t* calls, double* flops, double* bytes);

/* W[o, i] *= g[i], in place, rounded to the storage type: folds an RMSNorm gain g [in] into a
 * weight matrix [out, in] that consumes the normalised rows (pre-norm block placement; the
 * paper's Algorithm 1 leaves normalisation out). */
spts_status spts_fold_norm_gain(spts_ctx* ctx, void* W, const float* g, int out_features,
                                int in_features);

/* Partial Attention Probing, Eq. 4 / Algorithm 1 "K <- X W_K, q <- X_N W_Q; S_MHA":
 * K_out[n] = RoPE(rmsnorm(X[n]) W_K, pos[n]) for all N candidates (storage type, [N,Hkv,d]),
 * q = RoPE(rmsnorm(X[N-1]) W_Q, pos[N-1]),
 * S_mha_out[n] = (1/H) sum_h softmax_n(q_h . K_{h / (H/Hkv)} / sqrt(d))[n]   (fp32, [N]).
 * The logits are taken from the unrounded fp32 keys.  K_out may be NULL (workspace is used). */
spts_status spts_pap_score(spts_ctx* ctx, const spts_layer_weights* w, const void* X,
                           const int32_t* pos, int N, void* K_out, float* S_mha_out);

/* One-time repacking of a layer's proxy-FFN factors (Eq. 12) into the operand layouts the probe's GEMM chain reads,
 * so that nothing of it is left on the per-layer path: U_gate^T stacked over U_up^T (one [2r, D] matrix: the
 * residual stream is then read once for both), V_gate^T and V_up^T zero-padded to [D_low, 2r] each, and the Gram
 * matrix G = U_down^T U_down [r, r] split into a high and a low part: since ||t U_down^T||^2 = t G t^T, Eq. 13's
 * norm needs an [N, r] x [r, 2r] product instead of the [N, r] x [r, D] one.  `prepared` is caller-owned device
 * memory of spts_prepared_bytes(desc) bytes, 256-byte aligned; put its address into spts_layer_weights.prepared.
 * It must be redone when ug, uu, vg, vu or ud change.  Results are bit-identical with and without it. */
size_t spts_prepared_bytes(const spts_model_desc* desc);
spts_status spts_prepare_layer(spts_ctx* ctx, const spts_layer_weights* w, void* prepared, size_t prepared_bytes);

/* Low-rank Transformation Probing, Eq. 12-14: C[n] = || f(rmsnorm(X[n])) ||_2 with
 * f(x) = (silu(x Ug Vg) * (x Uu Vu)) Vd^T Ud^T, and S_ffn[n] = C[n] * S_mha[n].
 * C_out may be NULL.  X is the residual stream the FFN block would see. */
spts_status spts_ltp_score(spts_ctx* ctx, const spts_layer_weights* w, const void* X,
                           const float* S_mha, int N, float* C_out, float* S_ffn_out);

/* TopK of Eq. 5 / 15 / 16: the k largest of scores[0..N), written ascending by index.
 * Order: score descending, then index ascending; -0.0 equals +0.0; NaN ranks last (and sets
 * SPTS_ERR_NONFINITE in the device status).  flags: SPTS_FORCE_LAST.  1 <= k <= N. */
spts_status spts_topk_select(spts_ctx* ctx, const float* scores, int N, int k, uint32_t flags,
                             int32_t* idx_out);

/* The same selection for callers that cannot allocate device memory (the paper has no counterpart:
 * this exists for hosts whose device memory is planned and frozen before inference starts, or that are
 * only ever handed input and output buffers -- they can neither allocate the workspace spts_create()
 * needs nor let a library allocate behind their back).  It needs no context and no workspace: its
 * scratch is a fixed array of SPTS_TOPK_STATIC_SCRATCH_BYTES inside the library, resident on every GPU
 * that loads the library until the process exits.  Same result as spts_topk_select (same ordering rule,
 * ascending output, SPTS_FORCE_LAST); NaN scores rank last but are not reported, there being no context
 * to hold a status word.  Work is enqueued on `cuda_stream` (a cudaStream_t, may be 0) of the current
 * device and the call does not synchronise.
 *   - 1 <= k <= N <= SPTS_TOPK_STATIC_MAX_N, else SPTS_ERR_INVALID_ARG / SPTS_ERR_SHAPE before any launch.
 *   - The first call on each device looks up the array's device address (a synchronous runtime query,
 *     made with that device current); make that first call before any stream capture begins.
 *   - All calls on one device share the array.  Each call clears the counters it needs, so calls that
 *     are ordered on the GPU (same stream, or dependent streams) are fine; calls that may overlap on
 *     the GPU race on the scratch and give undefined index lists.
 *   - It calls no cudaMalloc / cudaFree or other allocating routine. */
#define SPTS_TOPK_STATIC_MAX_N 8388608
#define SPTS_TOPK_STATIC_SCRATCH_BYTES 36928
spts_status spts_topk_select_static(const float* scores, int N, int k, uint32_t flags, int32_t* idx_out,
                                    void* cuda_stream);

/* One decoder layer of Algorithm 1 in the prefill phase, in place on X [N, D]:
 *   S_mha (Eq. 4) -> T_a = TopK(S_mha, m_attn) -> Q, V projected for the rows in T_a, K rows
 *   reused -> cache <- (K^, V^, pos[T_a]) -> causal GQA attention among the active rows ->
 *   X[T_a] += O W_O (Eq. 2); then C, S_ffn (Eq. 12-14) on the updated X -> T_f =
 *   TopK(S_ffn, m_ffn) -> X[T_f] += FFN(rmsnorm(X[T_f])) (Eq. 6).  Rows outside T_a and T_f
 *   are not written.  m_attn == N / m_ffn == N run that block densely without probing.
 * cache->len is set to m_attn (capacity must be >= m_attn).  S_mha_out [N], idx_attn_out
 * [m_attn], idx_ffn_out [m_ffn] are optional outputs (NULL to skip; S_mha is still computed
 * when a selection needs it).  flags: SPTS_FORCE_LAST. */
spts_status spts_layer_prefill_skip(spts_ctx* ctx, const spts_layer_weights* w, void* X,
                                    const int32_t* pos, int N, int m_attn, int m_ffn,
                                    uint32_t flags, spts_kv_layer* cache, float* S_mha_out,
                                    int32_t* idx_attn_out, int32_t* idx_ffn_out);

/* The attention step of the reduced MHA on its own (Algorithm 1: O^ <- F_MHA(Q^, K^, V^), before W_O): causal
 * grouped-query attention among m rows in their compact order, row i attending to rows j <= i,
 *   O[i, h] = softmax_j(Q[i, h] . K[j, h / (H/Hkv)] / sqrt(d)) V[j, h / (H/Hkv)].
 * Q [m, H, d] and K [m, Hkv, d] are taken as given (after RoPE), V [m, Hkv, d]; O_out [m, H*d]; all in the storage
 * type, 16-byte aligned, none aliasing another.  1 <= m <= max_seq.  This is the kernel spts_layer_prefill_skip
 * runs between the Q/V projections and the O projection; the call exists so that it can be checked and timed on
 * operands of the caller's choosing. */
spts_status spts_reduced_attention(spts_ctx* ctx, const void* Q, const void* K, const void* V, int m, void* O_out);

/* The same layer for several independent prompts packed row after row into X [total, D] (the paper evaluates one
 * prompt at a time; Algorithm 1 applies to each prompt on its own, and that is what this call computes):
 * sequence b owns rows [seq_start[b], seq_start[b + 1]) of X and pos, has its own budgets m_attn[b], m_ffn[b]
 * (1 <= m <= its length) and its own cache caches[b].  seq_start [n_seq + 1], m_attn [n_seq], m_ffn [n_seq] and the
 * caches array are HOST memory; seq_start[0] == 0 and total = seq_start[n_seq] <= max_seq.
 * Everything that Eq. 4, 5 and 15 define per prompt stays per prompt: the probe uses each sequence's own last
 * token, its softmax runs over that sequence's candidates, TopK selects within the sequence (SPTS_FORCE_LAST keeps
 * each sequence's last row), attention is causal within the sequence.  The row normalisation, the K projection
 * (every row probed with its own sequence's last-token query), the per-sequence softmax and TopK, the Q / V / O
 * projections of all selected rows, the proxy FFN of Eq. 12-14 and the selected rows' SwiGLU FFN (Eq. 6) each run once
 * over the packed rows -- gathered GEMMs with ragged index lists, the attention kernel over a table of all
 * sequences' query tiles (tensor-core mode, up to 1024 sequences of up to 8192 rows each, probe window 1; other
 * batches run the attention blocks one sequence after the other).  Every row gets the bits the single-sequence call
 * gives it.
 * Optional outputs: S_mha_out [total]; idx_attn_out [sum m_attn] and idx_ffn_out [sum m_ffn], sequence after
 * sequence, each numbered from the sequence's own first row. */
spts_status spts_layer_prefill_skip_batch(spts_ctx* ctx, const spts_layer_weights* w, void* X, const int32_t* pos,
                                          int n_seq, const int32_t* seq_start, const int32_t* m_attn,
                                          const int32_t* m_ffn, uint32_t flags, spts_kv_layer* caches,
                                          float* S_mha_out, int32_t* idx_attn_out, int32_t* idx_ffn_out);

/* Stage-end pruning, Eq. 16 / Algorithm 1 "X <- X[T^{l+1}, :]": keeps the
 * n_next = min(N, N_{s+1}) candidates with the largest S_mha, in token order.  Out of place:
 * X_out [n_next, D], pos_out, orig_out [n_next] must not alias the inputs; idx_out [n_next]
 * (optional) receives the kept candidate indices.  flags: SPTS_FORCE_LAST. */
spts_status spts_msdp_compact(spts_ctx* ctx, const void* X_in, const int32_t* pos_in,
                              const int32_t* orig_in, const float* S_mha, int N, int n_next,
                              uint32_t flags, void* X_out, int32_t* pos_out, int32_t* orig_out,
                              int32_t* idx_out);

/* The budget rule of Multi-Stage Delayed Pruning (Section 3.4: M^l = min(|T^l|, M^l_fixed); Algorithm 1's
 * "M <- min(N, M_fix)" lines and the candidate update of Eq. 16), evaluated on the host: fills plan_out [n_layers]
 * (HOST memory) for a prompt of n_prompt tokens.  `stages` [n_stages] (HOST memory) is ordered by last_layer;
 * layer l belongs to the first stage whose last_layer >= l, layers after the last boundary to the last stage (they
 * keep its budgets).  Layers before `skip_from` run densely (m_attn = m_ffn = current candidate count) as the
 * paper's shallow layers do.  A stage's last layer gets prune_to = n_next when that is positive and smaller than
 * the current candidate count, and the later layers see that many candidates.  Optional outputs (host):
 * *n_final = candidates left after the last layer; *kv_token_layers = sum of m_attn over the layers, the number
 * of (token, layer) pairs the prefill leaves in the KV caches.  Pure host arithmetic: needs no context and no GPU.
 * Errors: SPTS_ERR_INVALID_ARG for null pointers, n_layers / n_prompt / n_stages < 1, stages out of order. */
spts_status spts_msdp_plan(int n_layers, int n_prompt, int skip_from, const spts_msdp_stage* stages, int n_stages,
                           spts_layer_plan* plan_out, int32_t* n_final, int64_t* kv_token_layers);

/* Offline construction of the low-rank proxy FFN of one layer (Section 3.3, "Low-rank Proxy FFN"):
 *   z(x) = |silu(x W_gate) * (x W_up)| for every calibration token x (rows of calib [n_cal, D], the hidden states
 *   preceding the FFN block, storage type; they are RMS-normalised like the FFN's input);
 *   I_j = mean of the max(1, floor(rho * n_cal)) largest z(x)[j] over the calibration tokens;
 *   C = TopK(I, D_low) (ascending, ties to the lower channel);  W' = W[:, C] for W_gate, W_up, W_down;
 *   W' ~ U V by truncated SVD of rank r (U has orthonormal columns, V carries the singular values).
 * Outputs, in the layouts spts_layer_weights expects (storage type): ug, uu [r, D]; vg, vu [D_low, r];
 * vd [r, D_low]; ud [D, r].  Optional: importance_out [Dff] fp32, channels_out [D_low] int32,
 * sigma_out [3, D_low] fp32 (singular values of the reduced gate, up, down matrices, descending).
 * `scratch` is caller-owned device memory of spts_proxy_scratch_bytes(desc, n_cal) bytes, 256-byte aligned.
 * Needs ltp_dlow <= ffn_dim, ltp_dlow even, ltp_rank <= min(ltp_dlow, hidden); 0 < rho <= 1.
 * Runs off the inference path (a few hundred small launches per matrix); asynchronous like every other call. */
size_t spts_proxy_scratch_bytes(const spts_model_desc* desc, int n_cal);
spts_status spts_proxy_build(spts_ctx* ctx, const spts_layer_weights* w, const void* calib, int n_cal, double rho,
                             void* scratch, size_t scratch_bytes, float* importance_out, int32_t* channels_out,
                             void* ug, void* vg, void* uu, void* vu, void* vd, void* ud, float* sigma_out);

/* End of prefill (the output of Algorithm 1 feeds next-token prediction): RMSNorm of one
 * hidden row x [D], logits = lm_head x (fp32 [vocab], optional), token = argmax (lowest index). */
spts_status spts_first_token(spts_ctx* ctx, const void* x_row, const void* lm_head,
                             float* logits_out, int32_t* token_out);

/* Whole prefill (Algorithm 1, prefill phase) over n_layers layers following `plan` (host
 * array [n_layers]).  X [N, D] is updated in place; at every stage end the survivors are
 * compacted into X_alt and the two buffers swap roles, likewise pos/orig with pos_alt/orig_alt
 * (each sized for N entries).  *n_final (host) receives the final candidate count and
 * *final_in_alt (host) tells which buffer holds the result.  token_out (device, optional)
 * receives the first generated token. */
spts_status spts_prefill(spts_ctx* ctx, const spts_model_weights* mw, const spts_layer_plan* plan,
                         void* X, int32_t* pos, int32_t* orig, void* X_alt, int32_t* pos_alt,
                         int32_t* orig_alt, int N, uint32_t flags, spts_kv_layer* caches,
                         int32_t* n_final, int32_t* final_in_alt, int32_t* token_out);

/* One decode step (Algorithm 1 outside the prefill phase: no skipping).  The new token's
 * embedding row is x_in [D] (if NULL, row token_in of mw->embed is used); it runs every layer
 * densely against that layer's cache plus itself at position `pos`, appends its K/V to every
 * cache (len += 1; capacity must allow it), then the first-token head.  x_out [D] optional. */
spts_status spts_decode_step(spts_ctx* ctx, const spts_model_weights* mw, spts_kv_layer* caches,
                             const void* x_in, int32_t token_in, int32_t pos, void* x_out,
                             float* logits_out, int32_t* token_out);

#ifdef __cplusplus
}
#endif
#endif /* SPTS_H_ */
