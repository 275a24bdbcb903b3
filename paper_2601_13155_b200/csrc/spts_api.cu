// C boundary of the SPTS library: argument checks, workspace carving and the per-layer
// schedule of Algorithm 1.  Everything here is host code that enqueues kernels on the context's
// stream; no call synchronises except spts_last_device_status().
#include <new>
#include <cmath>
#include <cstring>
#include <algorithm>
#include <vector>

#include "spts_common.cuh"

using namespace spts;

namespace {

// Hands out 256-byte aligned slices; every slice is followed by a guard band (GUARD_BYTES) whose offset is recorded.
struct Carver {
  char* base;
  size_t off;
  std::vector<size_t>* guards;
  template <typename T> T* take(size_t count) {
    off = align_up(off, 256);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off = align_up(off + count * sizeof(T), 256);
    if (guards) guards->push_back(off);
    off += GUARD_BYTES;
    return p;
  }
};

size_t elt_size(const spts_model_desc& d) { return d.dtype == SPTS_BF16 ? 2 : 4; }

// The SwiGLU intermediate [rows, Dff] is the widest buffer of a layer (28 KiB per row at the 8B shape).  The FFN block
// therefore runs over chunks of this many selected rows: per chunk the weights stream once more (a few hundred MB
// against ~6 TFLOP of work), and the workspace holds one chunk's intermediate instead of one row per candidate.
constexpr int FFN_CHUNK_ROWS = 16384;

bool shape_ok(const spts_model_desc& d) {
  if (d.hidden <= 0 || d.n_q_heads <= 0 || d.n_kv_heads <= 0 || d.ffn_dim <= 0) return false;
  if (d.n_q_heads % d.n_kv_heads != 0) return false;
  if (d.head_dim != 64 && d.head_dim != 128) return false;
  if (d.hidden % 8 || d.ffn_dim % 8 || d.ltp_dlow % 8 || d.ltp_rank % 8) return false;
  if (d.ltp_dlow <= 0 || d.ltp_rank <= 0) return false;
  if (d.dtype != SPTS_BF16 && d.dtype != SPTS_FP32) return false;
  if (d.n_layers <= 0) return false;
  return true;
}

// Shapes the tcgen05 kernels cover.
bool tc_shape_ok(const spts_model_desc& d) {
  return d.dtype == SPTS_BF16 && d.head_dim == 128 && d.hidden % 64 == 0 && d.ffn_dim % 64 == 0 &&
         d.ltp_dlow % 64 == 0 && d.ltp_rank % 16 == 0 && (d.n_q_heads * d.head_dim) % 64 == 0;
}

size_t carve(const spts_model_desc& d, int Nmax, void* base, Workspace* ws, std::vector<size_t>* guards = nullptr) {
  Carver c{reinterpret_cast<char*>(base), 0, guards};
  Workspace w;
  memset(&w, 0, sizeof(w));
  const size_t es = elt_size(d);
  const size_t N = (size_t)Nmax;
  const size_t HD = (size_t)d.n_q_heads * d.head_dim, KD = (size_t)d.n_kv_heads * d.head_dim;
  const size_t Npad = align_up(N, 128);
  w.status = c.take<int>(64);
  w.rstd = c.take<float>(N);
  w.q = c.take<float>(HD * (size_t)BATCH_MAX_SEQ);          // one probe query per sequence of a packed batch
  w.batch_i32 = c.take<int32_t>(6 * (size_t)(BATCH_MAX_SEQ + 1));
  w.batch_ptr = c.take<void*>(3 * (size_t)BATCH_MAX_SEQ);
  w.row_seq = c.take<int32_t>(N);
  w.vt_col = c.take<int32_t>(Npad);
  w.attn_tiles = c.take<int4>(Npad / 128 + (size_t)BATCH_MAX_SEQ);
  w.rope_cs = c.take<float2>(N * (d.head_dim / 2));
  w.vgu_pad = c.take<char>(2 * (size_t)d.ltp_dlow * 2 * d.ltp_rank * es);
  w.ugu = c.take<char>(2 * (size_t)d.ltp_rank * d.hidden * es);
  w.g2 = c.take<char>(2 * (size_t)d.ltp_rank * d.ltp_rank * es);
  {
    const size_t G = (size_t)d.n_q_heads / d.n_kv_heads;
    w.pw_logits = c.take<float>((size_t)PAP_MAX_WINDOW * G * Npad);
    w.pw_stats = c.take<float>(2 * (size_t)PAP_MAX_WINDOW * G);
    w.q_win = c.take<char>((size_t)PAP_MAX_WINDOW * HD * es);
    w.q_kv = c.take<char>((size_t)PAP_MAX_WINDOW * HD * es);
    w.idx_w = c.take<int32_t>(PAP_MAX_WINDOW);
  }
  w.logits = c.take<float>((size_t)d.n_q_heads * Npad);
  w.head_stats = c.take<float>(2 * (size_t)d.n_q_heads * BATCH_MAX_SEQ);
  w.s_mha = c.take<float>(N);
  w.s_ffn = c.take<float>(N);
  w.csq_parts = ceil_div(d.hidden, 64);
  w.csq = c.take<float>(N * w.csq_parts);
  w.idx_a = c.take<int32_t>(Npad);
  w.idx_f = c.take<int32_t>(Npad);
  w.idx_p = c.take<int32_t>(Npad);
  w.topk_scratch = c.take<uint32_t>(TOPK_SCRATCH_WORDS);
  w.k_all = c.take<char>(N * KD * es);
  w.q_act = c.take<char>(Npad * HD * es);
  w.vt_ld_max = (int)(Npad + 8 * (size_t)BATCH_MAX_SEQ);     // a packed batch starts every sequence's columns on a multiple of 8
  w.v_t = c.take<char>(KD * (size_t)w.vt_ld_max * es);
  w.o_att = c.take<char>(Npad * HD * es);
  w.hm = c.take<char>((Npad < (size_t)FFN_CHUNK_ROWS ? Npad : (size_t)FFN_CHUNK_ROWS) * (size_t)d.ffn_dim * es);
  w.t1 = c.take<char>(Npad * 2 * (size_t)d.ltp_rank * es);
  w.hlow = c.take<char>(Npad * (size_t)d.ltp_dlow * es);
  w.t2 = c.take<char>(Npad * (size_t)d.ltp_rank * es);
  // The fp32 keys of the plain-kernel K projection live only between that GEMM and the logits kernel behind it, when
  // the attention output buffer of the block is still unused: they share its storage whenever it is large enough.
  w.acc32_elems = N * KD;
  if (Npad * HD * es >= w.acc32_elems * sizeof(float)) w.acc32 = reinterpret_cast<float*>(w.o_att);
  else w.acc32 = c.take<float>(w.acc32_elems);
  w.dec = c.take<float>(decode_scratch_floats(d));
  w.logits_v = c.take<float>((size_t)(d.vocab > 0 ? d.vocab : 1));
  w.xrow = c.take<char>((size_t)d.hidden * es);
  if (ws) *ws = w;
  return align_up(c.off, 256);
}

bool use_tc(const spts_ctx* ctx) { return ctx->desc.dtype == SPTS_BF16 && !ctx->reference_kernels; }

// One GEMM with fused epilogue on whichever kernel family the context uses.
struct Gemm {
  const void* A; int lda; int a_rows;
  const int32_t* idx; const int32_t* dst_idx;
  const void* W; const void* W2;
  int M, Nout, K;
  const float* rowscale;
  void* out; int ldo;
  void* out_t; int ldt;
  const float* q; float* logits; int ld_logits;
  float* csq;
  float* sal_t; int ld_sal;
  int ldw; float* out_f32;
};

spts_status run_gemm(spts_ctx* ctx, int epi, const Gemm& g) {
  if (g.M <= 0) return SPTS_OK;
  const auto& d = ctx->desc;
  if (use_tc(ctx)) {
    TcGemmArgs a;
    memset(&a, 0, sizeof(a));
    a.A = (const bf16*)g.A; a.lda = g.lda; a.a_rows = g.a_rows; a.idx = g.idx; a.dst_idx = g.dst_idx;
    a.W = (const bf16*)g.W; a.W2 = (const bf16*)g.W2; a.M = g.M; a.Nout = g.Nout; a.K = g.K;
    a.rowscale = g.rowscale; a.out = (bf16*)g.out; a.ldo = g.ldo; a.out_t = (bf16*)g.out_t; a.ldt = g.ldt;
    a.q = g.q; a.logits = g.logits; a.ld_logits = g.ld_logits; a.group = d.n_q_heads / d.n_kv_heads;
    a.csq = g.csq; a.csq_parts = ctx->ws.csq_parts; a.sal_t = g.sal_t; a.ld_sal = g.ld_sal;
    a.ldw = g.ldw; a.out_f32 = g.out_f32;
    return launch_tc_gemm(ctx, epi, a);
  }
  RefGemmArgs a;
  memset(&a, 0, sizeof(a));
  a.A = g.A; a.lda = g.lda; a.idx = g.idx; a.dst_idx = g.dst_idx; a.W = g.W; a.W2 = g.W2;
  a.M = g.M; a.Nout = g.Nout; a.K = g.K; a.rowscale = g.rowscale; a.out = g.out; a.ldo = g.ldo;
  a.out_t = g.out_t; a.ldt = g.ldt; a.head_dim = d.head_dim; a.q = g.q; a.logits = g.logits;
  a.ld_logits = g.ld_logits; a.group = d.n_q_heads / d.n_kv_heads; a.csq = g.csq; a.csq_parts = ctx->ws.csq_parts;
  a.sal_t = g.sal_t; a.ld_sal = g.ld_sal; a.ldw = g.ldw; a.out_f32 = g.out_f32;
  return launch_ref_gemm(ctx, epi, a);
}

#define TRY(x) do { spts_status s__ = (x); if (s__ != SPTS_OK) return s__; } while (0)

// ---- optional per-operation timing with CUDA events on the context's stream
struct ProfRecord { cudaEvent_t a, b; int tag; double flops, bytes; };
struct Profiler {
  int filter = 0;                 // 0 off, -1 every operation, else one SPTS_OP_* tag
  std::vector<ProfRecord> recs;
  std::vector<cudaEvent_t> pool;
  size_t used = 0;
  cudaEvent_t get() {
    if (used == pool.size()) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
      pool.push_back(e);
    }
    return pool[used++];
  }
};
Profiler* prof_of(spts_ctx* ctx) { return reinterpret_cast<Profiler*>(ctx->prof); }

struct ProfScope {
  spts_ctx* ctx; ProfRecord r; bool on;
  ProfScope(spts_ctx* c, int tag, double flops, double bytes) : ctx(c), on(false) {
    Profiler* p = prof_of(c);
    if (p == nullptr || p->filter == 0 || (p->filter != -1 && p->filter != tag) || p->recs.size() >= 65536) return;
    r.a = p->get(); r.b = p->get();
    if (r.a == nullptr || r.b == nullptr) return;
    r.tag = tag; r.flops = flops; r.bytes = bytes;
    on = cudaEventRecord(r.a, c->stream) == cudaSuccess;
  }
  ~ProfScope() {
    if (on && cudaEventRecord(r.b, ctx->stream) == cudaSuccess) prof_of(ctx)->recs.push_back(r);
  }
};
#define OP(tag, flops, bytes, call) do { ProfScope ps__(ctx, tag, flops, bytes); TRY(call); } while (0)

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Probe score averaged over the last `window` queries (the query-length ablation of the paper's Appendix C):
// S_n = 1 / (window * H) * sum_i sum_h softmax_{n <= i}(q_{i,h} . K_n / sqrt(d)), each query over its causal range.
// rstd and the rotary table are ready.  K and the window's queries are taken as stored (rounded to the storage
// type); the logits of one KV head's queries against all keys are one small GEMM with fp32 output.
spts_status pap_window_tail(spts_ctx* ctx, const spts_layer_weights* w, const void* X, int N, void* K_out, int window,
                            float* S_out) {
  const auto& d = ctx->desc;
  Workspace& ws = ctx->ws;
  const int HD = d.n_q_heads * d.head_dim, KD = d.n_kv_heads * d.head_dim, G = d.n_q_heads / d.n_kv_heads;
  const int ld = (int)align_up((size_t)N, 128);
  const size_t es = elt_size(d);
  const double Nd = (double)N, Dd = (double)d.hidden;
  Gemm g;
  memset(&g, 0, sizeof(g));
  g.A = X; g.lda = d.hidden; g.a_rows = N; g.W = w->wk; g.M = N; g.Nout = KD; g.K = d.hidden;
  g.rowscale = ws.rstd; g.out = K_out; g.ldo = KD;
  OP(SPTS_OP_KPROJ, 2.0 * Nd * Dd * KD, (Nd * Dd + Nd * KD + Dd * KD) * es, run_gemm(ctx, REF_ROPE, g));
  ProfScope ps(ctx, SPTS_OP_PAP_SOFTMAX, 2.0 * Nd * window * HD + 2.0 * window * Dd * HD,
               (Nd * KD + window * Dd) * es + 8.0 * Nd * window * d.n_q_heads);
  TRY(launch_iota_from(ctx, ws.idx_w, window, N - window));
  memset(&g, 0, sizeof(g));
  g.A = X; g.lda = d.hidden; g.a_rows = N; g.idx = ws.idx_w; g.W = w->wq; g.M = window; g.Nout = HD; g.K = d.hidden;
  g.rowscale = ws.rstd; g.out = ws.q_win; g.ldo = HD;
  TRY(run_gemm(ctx, REF_ROPE, g));
  TRY(launch_pap_regroup(ctx, ws.q_win, window, ws.q_kv));
  for (int kvh = 0; kvh < d.n_kv_heads; ++kvh) {
    memset(&g, 0, sizeof(g));
    g.A = (const char*)ws.q_kv + (size_t)kvh * window * G * d.head_dim * es; g.lda = d.head_dim; g.a_rows = window * G;
    g.W = (const char*)K_out + (size_t)kvh * d.head_dim * es; g.ldw = KD;
    g.M = window * G; g.Nout = N; g.K = d.head_dim; g.out_f32 = ws.pw_logits; g.ldo = ld;
    TRY(run_gemm(ctx, REF_STORE, g));
    TRY(launch_pap_window_softmax(ctx, ws.pw_logits, ld, N, window, kvh > 0 ? 1 : 0, ws.pw_stats, S_out));
  }
  return SPTS_OK;
}

// PAP (Eq. 4): rstd, rotary table, q of the last row, K of every row with the logits taken from
// the unrounded keys in the projection's epilogue, then the head-mean softmax.
spts_status pap_pipeline(spts_ctx* ctx, const spts_layer_weights* w, const void* X, const int32_t* pos, int N,
                         void* K_out, bool want_scores, float* S_out) {
  const auto& d = ctx->desc;
  Workspace& ws = ctx->ws;
  const int KD = d.n_kv_heads * d.head_dim;
  const int ld = (int)align_up((size_t)N, 128);
  const double es = (double)elt_size(d), Nd = (double)N, Dd = (double)d.hidden;
  if (ctx->rstd_rows != nullptr && ctx->rstd_x == X && ctx->rstd_n == N) {
    // inside spts_prefill: only the rows the previous layer's FFN block updated have a new statistic
    OP(SPTS_OP_PREP, 0.0, ctx->rstd_nrows * (Dd * es + 8.0), launch_rstd_rows(ctx, X, ctx->rstd_rows, ctx->rstd_nrows, ws.rstd));
  } else {
    OP(SPTS_OP_PREP, 0.0, Nd * Dd * es + 4.0 * Nd, launch_rstd(ctx, X, N, ws.rstd));
  }
  ctx->rstd_rows = nullptr;
  if (!(ctx->rope_trust && ctx->rope_pos == pos && ctx->rope_n == N)) {
    OP(SPTS_OP_PREP, 0.0, Nd * (4.0 + 4.0 * d.head_dim), launch_rope_table(ctx, pos, N, ws.rope_cs));
    ctx->rope_pos = pos;
    ctx->rope_n = N;
  }
  if (want_scores && (ctx->pap_window < 2 || N < 2))
    OP(SPTS_OP_PREP, 2.0 * Dd * d.n_q_heads * d.head_dim, Dd * d.n_q_heads * d.head_dim * es,
       launch_q_last(ctx, X, ws.rope_cs, N, w->wq, ws.rstd, ws.q));
  const int window = ctx->pap_window < N ? ctx->pap_window : N;
  if (want_scores && window > 1) return pap_window_tail(ctx, w, X, N, K_out, window, S_out);
  Gemm g;
  memset(&g, 0, sizeof(g));
  g.A = X; g.lda = d.hidden; g.a_rows = N; g.W = w->wk; g.M = N; g.Nout = KD; g.K = d.hidden;
  g.rowscale = ws.rstd; g.out = K_out; g.ldo = KD;
  if (want_scores) { g.q = ws.q; g.logits = ws.logits; g.ld_logits = ld; }
  OP(SPTS_OP_KPROJ, 2.0 * Nd * Dd * KD, (Nd * Dd + Nd * KD + Dd * KD) * es, run_gemm(ctx, REF_ROPE, g));
  if (want_scores)
    OP(SPTS_OP_PAP_SOFTMAX, 0.0, Nd * 4.0 * (2.0 * d.n_q_heads + 1.0), launch_pap_softmax(ctx, ws.logits, ld, N, S_out));
  return SPTS_OK;
}

// Layout of a prepared-layer buffer (spts_prepare_layer): [Ug^T ; Uu^T] [2r, D], then [Vg^T | 0] and [0 | Vu^T]
// ([D_low, 2r] each), then [G_hi ; G_lo] [2r, r] (tensor-core mode), each slice 256-byte aligned.
struct PreparedLayout { size_t ugu, vgu, g2, total; };
PreparedLayout prepared_layout(const spts_model_desc& d) {
  const size_t es = elt_size(d);
  PreparedLayout l;
  l.ugu = 0;
  l.vgu = align_up(l.ugu + 2 * (size_t)d.ltp_rank * d.hidden * es, 256);
  l.g2 = align_up(l.vgu + 2 * (size_t)d.ltp_dlow * 2 * d.ltp_rank * es, 256);
  l.total = align_up(l.g2 + 2 * (size_t)d.ltp_rank * d.ltp_rank * es, 256);
  return l;
}

// Eq. 13 as a quadratic form in the Gram matrix of U_down: tensor-core mode with a rank the epilogue's 32-column
// chunks divide.  Otherwise the proxy output's sum of squares is taken from the [N, r] x [r, D] product itself.
bool ltp_uses_gram(const spts_ctx* ctx) { return use_tc(ctx) && ctx->desc.ltp_rank % 32 == 0; }

spts_status pack_proxy(spts_ctx* ctx, const spts_layer_weights* w, void* ugu, void* vgu, void* g2) {
  const auto& d = ctx->desc;
  const size_t ubytes = (size_t)d.ltp_rank * d.hidden * elt_size(d);
  TRY(launch_pad_proxy(ctx, w->vg, w->vu, vgu));
  if (cudaMemcpyAsync(ugu, w->ug, ubytes, cudaMemcpyDeviceToDevice, ctx->stream) != cudaSuccess ||
      cudaMemcpyAsync((char*)ugu + ubytes, w->uu, ubytes, cudaMemcpyDeviceToDevice, ctx->stream) != cudaSuccess)
    return SPTS_ERR_CUDA;
  if (ltp_uses_gram(ctx)) TRY(launch_gram(ctx, w->ud, g2));
  return SPTS_OK;
}

// LTP (Eq. 12-14) on rows already normalised through `rstd`.
spts_status ltp_pipeline(spts_ctx* ctx, const spts_layer_weights* w, const void* X, const float* S_mha, int N,
                         float* C_out, float* S_ffn_out) {
  const auto& d = ctx->desc;
  Workspace& ws = ctx->ws;
  const int r = d.ltp_rank, Dl = d.ltp_dlow;
  const size_t es = elt_size(d);
  const double Nd = (double)N;
  ProfScope ps_ltp(ctx, SPTS_OP_LTP, 6.0 * Nd * r * ((double)d.hidden + Dl),
                   Nd * d.hidden * (double)es + 3.0 * r * ((double)d.hidden + Dl) * (double)es + 8.0 * Nd);
  // the repacked factors: the layer's prepared buffer, or packed here into the workspace
  const void* ugu = ws.ugu; const void* vgu = ws.vgu_pad; const void* g2 = ws.g2;
  if (w->prepared != nullptr) {
    const PreparedLayout pl = prepared_layout(d);
    const char* base = (const char*)w->prepared;
    ugu = base + pl.ugu; vgu = base + pl.vgu; g2 = base + pl.g2;
  } else {
    TRY(pack_proxy(ctx, w, ws.ugu, ws.vgu_pad, ws.g2));
  }
  Gemm g;
  // t1 = [x Ug | x Uu]: the two first factors are stacked into one [2r, D] matrix so that the residual
  // stream (the only large operand of the whole proxy) is read once
  memset(&g, 0, sizeof(g));
  g.A = X; g.lda = d.hidden; g.a_rows = N; g.W = ugu; g.M = N; g.Nout = 2 * r; g.K = d.hidden;
  g.rowscale = ws.rstd; g.out = ws.t1; g.ldo = 2 * r;
  TRY(run_gemm(ctx, REF_STORE, g));
  // hlow = silu(t_g Vg) * (t_u Vu)
  memset(&g, 0, sizeof(g));
  g.A = ws.t1; g.lda = 2 * r; g.a_rows = N; g.W = vgu; g.W2 = (const char*)vgu + (size_t)Dl * 2 * r * es;
  g.M = N; g.Nout = Dl; g.K = 2 * r; g.out = ws.hlow; g.ldo = Dl;
  TRY(run_gemm(ctx, REF_SWIGLU, g));
  // t2 = hlow Vd^T
  memset(&g, 0, sizeof(g));
  g.A = ws.hlow; g.lda = Dl; g.a_rows = N; g.W = w->vd; g.M = N; g.Nout = r; g.K = Dl; g.out = ws.t2; g.ldo = r;
  TRY(run_gemm(ctx, REF_STORE, g));
  int parts;
  memset(&g, 0, sizeof(g));
  if (ltp_uses_gram(ctx)) {
    // C^2 = t2 G t2^T with G = Ud^T Ud: y = t2 [G_hi ; G_lo]^T, and the epilogue dots y with the row of t2 itself
    g.A = ws.t2; g.lda = r; g.a_rows = N; g.W = g2; g.M = N; g.Nout = 2 * r; g.K = r; g.csq = ws.csq;
    TRY(run_gemm(ctx, TC_QFORM, g));
    parts = ceil_div(2 * r, 256);
  } else {
    // C^2 = || t2 Ud^T ||^2, summed in the epilogue
    g.A = ws.t2; g.lda = r; g.a_rows = N; g.W = w->ud; g.M = N; g.Nout = d.hidden; g.K = r; g.csq = ws.csq;
    TRY(run_gemm(ctx, REF_SUMSQ, g));
    parts = use_tc(ctx) ? tc_sumsq_parts(d.hidden) : ceil_div(d.hidden, 64);
  }
  TRY(launch_ffn_score(ctx, ws.csq, parts, S_mha, N, C_out, S_ffn_out));
  return SPTS_OK;
}

// PAP + reduced MHA of one sequence (Eq. 4, 5, Eq. 2 for the attention block): X rows updated in place, cache filled.
// want_scores: S is needed later (FFN selection or the caller asked for it).
spts_status attention_block(spts_ctx* ctx, const spts_layer_weights* w, void* X, const int32_t* pos, int N, int m_attn,
                            bool want_scores_later, uint32_t flags, spts_kv_layer* cache, float* S,
                            int32_t* idx_attn_out) {
  const auto& d = ctx->desc;
  Workspace& ws = ctx->ws;
  const int D = d.hidden, HD = d.n_q_heads * d.head_dim, KD = d.n_kv_heads * d.head_dim;
  const size_t es = elt_size(d);
  const bool sel_a = m_attn < N;
  const bool want_scores = sel_a || want_scores_later;
  const bool tc = use_tc(ctx);

  // ---- PAP + reduced MHA
  void* k_dst = sel_a ? ws.k_all : cache->k;
  TRY(pap_pipeline(ctx, w, X, pos, N, k_dst, want_scores, S));
  const int32_t* idx_a = nullptr;
  if (sel_a) {
    int32_t* ia = idx_attn_out ? idx_attn_out : ws.idx_a;
    OP(SPTS_OP_TOPK, 0.0, 4.0 * N + 4.0 * m_attn, launch_topk(ctx, S, N, m_attn, flags, ia, ws.topk_scratch));
    if (ctx->debug_checks) TRY(launch_check_index_list(ctx, ia, m_attn, N));
    OP(SPTS_OP_KV_GATHER, 0.0, 2.0 * m_attn * (double)KD * es + 8.0 * m_attn,
       launch_gather_rows(ctx, ws.k_all, ia, m_attn, (int)(KD * es), cache->k));
    OP(SPTS_OP_KV_GATHER, 0.0, 12.0 * m_attn, launch_gather_i32(ctx, pos, ia, m_attn, cache->pos));
    idx_a = ia;
  } else {
    if (cudaMemcpyAsync(cache->pos, pos, (size_t)N * sizeof(int32_t), cudaMemcpyDeviceToDevice, ctx->stream) != cudaSuccess)
      return SPTS_ERR_CUDA;
    if (idx_attn_out) TRY(launch_topk(ctx, S, N, N, flags, idx_attn_out, ws.topk_scratch));
  }
  const int ldvt = (int)align_up((size_t)m_attn, 128);
  Gemm g;
  memset(&g, 0, sizeof(g));
  g.A = X; g.lda = D; g.a_rows = N; g.idx = idx_a; g.W = w->wq; g.M = m_attn; g.Nout = HD; g.K = D;
  g.rowscale = ws.rstd; g.out = ws.q_act; g.ldo = HD;
  const double Ma = (double)m_attn, Dd = (double)D, esd = (double)es;
  OP(SPTS_OP_QVPROJ, 2.0 * Ma * Dd * HD, (Ma * Dd + Ma * HD + Dd * HD) * esd, run_gemm(ctx, REF_ROPE, g));
  g.W = w->wv; g.Nout = KD; g.out = cache->v; g.ldo = KD;
  if (tc) { g.out_t = ws.v_t; g.ldt = ldvt; }
  OP(SPTS_OP_QVPROJ, 2.0 * Ma * Dd * KD, (Ma * Dd + 2.0 * Ma * KD + Dd * KD) * esd, run_gemm(ctx, REF_STORE, g));
  ProfScope* ps_att = new ProfScope(ctx, SPTS_OP_ATTN, 2.0 * HD * Ma * (Ma + 1.0), (2.0 * Ma * HD + 2.0 * Ma * KD) * esd);
  spts_status s_att = SPTS_OK;
  if (tc) s_att = (launch_tc_attention(ctx, (const bf16*)ws.q_act, (const bf16*)cache->k, (const bf16*)cache->v, (const bf16*)ws.v_t, ldvt, m_attn,
                                  (bf16*)ws.o_att));
  else s_att = launch_ref_attention(ctx, ws.q_act, cache->k, cache->v, m_attn, ws.o_att);
  delete ps_att;
  TRY(s_att);
  memset(&g, 0, sizeof(g));
  g.A = ws.o_att; g.lda = HD; g.a_rows = m_attn; g.dst_idx = idx_a; g.W = w->wo; g.M = m_attn; g.Nout = D; g.K = HD;
  g.out = X; g.ldo = D;
  OP(SPTS_OP_OPROJ, 2.0 * Ma * Dd * HD, (Ma * HD + 2.0 * Ma * Dd + Dd * HD) * esd, run_gemm(ctx, REF_RESID, g));
  cache->len = m_attn;

  return SPTS_OK;
}

// SwiGLU FFN on the rows `idx_f` (nullptr: all a_rows rows) of X with the residual scatter (Eq. 6, Eq. 2); X is
// normalised through ws.rstd
spts_status ffn_gemms(spts_ctx* ctx, const spts_layer_weights* w, void* X, int N, const int32_t* idx_f, int m_ffn) {
  const auto& d = ctx->desc;
  Workspace& ws = ctx->ws;
  const int D = d.hidden;
  const double Dd = (double)D, esd = (double)elt_size(d);
  const size_t row_bytes = (size_t)D * elt_size(d);
  for (int c0 = 0; c0 < m_ffn; c0 += FFN_CHUNK_ROWS) {
    const int mc = m_ffn - c0 < FFN_CHUNK_ROWS ? m_ffn - c0 : FFN_CHUNK_ROWS;
    const double Mf = (double)mc;
    // without an index list the chunk is rows [c0, c0 + mc) of X itself
    char* xc = idx_f ? (char*)X : (char*)X + (size_t)c0 * row_bytes;
    const int32_t* ic = idx_f ? idx_f + c0 : nullptr;
    Gemm g;
    memset(&g, 0, sizeof(g));
    g.A = xc; g.lda = D; g.a_rows = idx_f ? N : mc; g.idx = ic; g.W = w->w_gate; g.W2 = w->w_up; g.M = mc; g.Nout = d.ffn_dim;
    g.K = D; g.rowscale = idx_f ? ws.rstd : ws.rstd + c0; g.out = ws.hm; g.ldo = d.ffn_dim;
    OP(SPTS_OP_GATEUP, 4.0 * Mf * Dd * d.ffn_dim, (Mf * Dd + Mf * d.ffn_dim + 2.0 * Dd * d.ffn_dim) * esd,
       run_gemm(ctx, REF_SWIGLU, g));
    memset(&g, 0, sizeof(g));
    g.A = ws.hm; g.lda = d.ffn_dim; g.a_rows = mc; g.dst_idx = ic; g.W = w->w_down; g.M = mc; g.Nout = D;
    g.K = d.ffn_dim; g.out = xc; g.ldo = D;
    OP(SPTS_OP_DOWN, 2.0 * Mf * Dd * d.ffn_dim, (Mf * d.ffn_dim + 2.0 * Mf * Dd + Dd * d.ffn_dim) * esd,
       run_gemm(ctx, REF_RESID, g));
  }
  return SPTS_OK;
}

// The attention blocks of a packed batch with one launch per step instead of one per step and sequence (tensor-core
// mode, probe window 1, at most BATCH_MAX_SEQ sequences of at most TOPK_SEG_MAX rows): the row statistics, the
// rotary table, every sequence's last-token query, the K projection with each row probed by its own sequence's
// query, the per-sequence softmax of Eq. 4 and TopK of Eq. 5, the Q / V projections of all selected rows and the O
// projection run once over the packed rows, and the causal attention of all sequences is one launch over a table
// of their query tiles.  Every row gets the bits the single-sequence call gives it.
spts_status batch_attention_blocks(spts_ctx* ctx, const spts_layer_weights* w, void* X, const int32_t* pos, int n_seq,
                                   const int32_t* seq_start, const int32_t* m_attn, uint32_t flags, spts_kv_layer* caches,
                                   float* S, int32_t* idx_attn_out) {
  const auto& d = ctx->desc;
  Workspace& ws = ctx->ws;
  const int D = d.hidden, HD = d.n_q_heads * d.head_dim, KD = d.n_kv_heads * d.head_dim;
  const int total = seq_start[n_seq];
  const size_t es = elt_size(d);
  // host tables: seq_start | m_attn | act_off | vt0, and the caches' pointers
  std::vector<int32_t> tab((size_t)4 * (n_seq + 1), 0);
  int32_t* h_start = tab.data();
  int32_t* h_m = h_start + (n_seq + 1);
  int32_t* h_off = h_m + (n_seq + 1);
  int32_t* h_vt0 = h_off + (n_seq + 1);
  std::vector<void*> ptrs((size_t)3 * n_seq);
  int A = 0, vt = 0, max_len = 0;
  for (int b = 0; b < n_seq; ++b) {
    h_start[b] = seq_start[b]; h_m[b] = m_attn[b]; h_off[b] = A; h_vt0[b] = vt;
    A += m_attn[b];
    vt += (m_attn[b] + 7) & ~7;
    const int len = seq_start[b + 1] - seq_start[b];
    max_len = len > max_len ? len : max_len;
    ptrs[b] = caches[b].k; ptrs[n_seq + b] = caches[b].v; ptrs[2 * n_seq + b] = caches[b].pos;
  }
  h_start[n_seq] = total; h_off[n_seq] = A;
  const int ldvt = (int)align_up((size_t)vt, 128);
  if (ldvt > ws.vt_ld_max) return SPTS_ERR_WORKSPACE;
  int32_t* d_start = ws.batch_i32;
  int32_t* d_m = d_start + (n_seq + 1);
  int32_t* d_off = d_m + (n_seq + 1);
  int32_t* d_vt0 = d_off + (n_seq + 1);
  if (cudaMemcpyAsync(d_start, tab.data(), tab.size() * sizeof(int32_t), cudaMemcpyHostToDevice, ctx->stream) != cudaSuccess ||
      cudaMemcpyAsync(ws.batch_ptr, ptrs.data(), ptrs.size() * sizeof(void*), cudaMemcpyHostToDevice, ctx->stream) != cudaSuccess)
    return SPTS_ERR_CUDA;
  const double Nd = (double)total, Dd = (double)D, esd = (double)es, Ad = (double)A;
  const int ld = (int)align_up((size_t)total, 128);
  // ---- probe (Eq. 4), per sequence
  OP(SPTS_OP_PREP, 0.0, Nd * Dd * esd + 4.0 * Nd, launch_rstd(ctx, X, total, ws.rstd));
  ctx->rope_trust = false;
  OP(SPTS_OP_PREP, 0.0, Nd * (4.0 + 4.0 * d.head_dim), launch_rope_table(ctx, pos, total, ws.rope_cs));
  TRY(launch_batch_row_seq(ctx, d_start, n_seq, total, ws.row_seq));
  OP(SPTS_OP_PREP, 2.0 * n_seq * Dd * HD, Dd * HD * esd, launch_q_last_batch(ctx, X, ws.rope_cs, d_start, n_seq, w->wq, ws.rstd, ws.q));
  {
    TcGemmArgs a;
    memset(&a, 0, sizeof(a));
    a.A = (const bf16*)X; a.lda = D; a.a_rows = total; a.W = (const bf16*)w->wk; a.M = total; a.Nout = KD; a.K = D;
    a.rowscale = ws.rstd; a.out = (bf16*)ws.k_all; a.ldo = KD; a.q = ws.q; a.logits = ws.logits; a.ld_logits = ld;
    a.group = d.n_q_heads / d.n_kv_heads; a.row_seq = ws.row_seq; a.q_stride = HD; a.csq_parts = ws.csq_parts;
    OP(SPTS_OP_KPROJ, 2.0 * Nd * Dd * KD, (Nd * Dd + Nd * KD + Dd * KD) * esd, launch_tc_gemm(ctx, TC_ROPE, a));
  }
  OP(SPTS_OP_PAP_SOFTMAX, 0.0, Nd * 4.0 * (2.0 * d.n_q_heads + 1.0),
     launch_pap_softmax_batch(ctx, ws.logits, ld, d_start, n_seq, total, ws.row_seq, ws.head_stats, S));
  // ---- TopK (Eq. 5) per sequence: lists numbered within the sequence for the caller, within the batch for the gathers
  OP(SPTS_OP_TOPK, 0.0, 4.0 * Nd + 4.0 * Ad,
     launch_topk_segmented(ctx, S, d_start, d_m, d_off, n_seq, max_len, flags, idx_attn_out, ws.idx_a));
  if (ctx->debug_checks) TRY(launch_check_index_list(ctx, ws.idx_a, A, total));
  TRY(launch_batch_vt_col(ctx, d_off, d_vt0, n_seq, A, ws.vt_col));
  // ---- Q and V of the selected rows; V goes through the (still unused) attention-output buffer to the caches
  {
    TcGemmArgs a;
    memset(&a, 0, sizeof(a));
    a.A = (const bf16*)X; a.lda = D; a.a_rows = total; a.idx = ws.idx_a; a.W = (const bf16*)w->wq; a.M = A; a.Nout = HD; a.K = D;
    a.rowscale = ws.rstd; a.out = (bf16*)ws.q_act; a.ldo = HD; a.group = d.n_q_heads / d.n_kv_heads; a.csq_parts = ws.csq_parts;
    OP(SPTS_OP_QVPROJ, 2.0 * Ad * Dd * HD, (Ad * Dd + Ad * HD + Dd * HD) * esd, launch_tc_gemm(ctx, TC_ROPE, a));
    // a prompt's last key block reaches into the columns after its own: the up to seven pad columns before the next
    // prompt's start must hold finite values (they meet probabilities that are exactly zero)
    if (cudaMemsetAsync(ws.v_t, 0, (size_t)KD * ldvt * es, ctx->stream) != cudaSuccess) return SPTS_ERR_CUDA;
    a.W = (const bf16*)w->wv; a.Nout = KD; a.out = (bf16*)ws.o_att; a.ldo = KD;
    a.out_t = (bf16*)ws.v_t; a.ldt = ldvt; a.out_t_col = ws.vt_col;
    OP(SPTS_OP_QVPROJ, 2.0 * Ad * Dd * KD, (Ad * Dd + 2.0 * Ad * KD + Dd * KD) * esd, launch_tc_gemm(ctx, TC_STORE, a));
  }
  OP(SPTS_OP_KV_GATHER, 0.0, 4.0 * Ad * (double)KD * esd + 12.0 * Ad,
     launch_batch_cache_fill(ctx, ws.k_all, ws.o_att, pos, ws.idx_a, d_off, n_seq, A, ws.batch_ptr, ws.batch_ptr + n_seq,
                             (int32_t* const*)(ws.batch_ptr + 2 * n_seq)));
  // ---- causal attention of every prompt among its own active rows (Algorithm 1: F_MHA(Q^, K^, V^)) in one launch:
  //      K^ packed like Q^ (in the FFN intermediate's buffer, idle during the attention block), a table of the
  //      prompts' query tiles, longest first
  {
    const bool pair_tiles = (d.n_q_heads / d.n_kv_heads) % 2 != 0;
    std::vector<int4> tiles;
    for (int b = 0; b < n_seq; ++b) {
      const int nqt = ceil_div(m_attn[b], 128), ny = pair_tiles ? ceil_div(nqt, 2) : nqt;
      for (int y = 0; y < ny; ++y) tiles.push_back(make_int4(h_off[b], h_vt0[b], m_attn[b], y));
    }
    std::stable_sort(tiles.begin(), tiles.end(), [](const int4& a, const int4& b) { return a.w > b.w; });
    if (cudaMemcpyAsync(ws.attn_tiles, tiles.data(), tiles.size() * sizeof(int4), cudaMemcpyHostToDevice, ctx->stream) != cudaSuccess)
      return SPTS_ERR_CUDA;
    OP(SPTS_OP_KV_GATHER, 0.0, 2.0 * Ad * (double)KD * esd, launch_gather_rows(ctx, ws.k_all, ws.idx_a, A, (int)(KD * es), ws.hm));
    double fl = 0.0;
    for (int b = 0; b < n_seq; ++b) fl += 2.0 * HD * (double)m_attn[b] * (m_attn[b] + 1.0);
    OP(SPTS_OP_ATTN, fl, (2.0 * Ad * HD + 2.0 * Ad * KD) * esd,
       launch_tc_attention_packed(ctx, (const bf16*)ws.q_act, (const bf16*)ws.hm, (const bf16*)ws.v_t, ldvt, A, vt,
                                  ws.attn_tiles, (int)tiles.size(), (bf16*)ws.o_att));
  }
  {
    TcGemmArgs a;
    memset(&a, 0, sizeof(a));
    a.A = (const bf16*)ws.o_att; a.lda = HD; a.a_rows = A; a.dst_idx = ws.idx_a; a.W = (const bf16*)w->wo; a.M = A; a.Nout = D; a.K = HD;
    a.out = (bf16*)X; a.ldo = D; a.csq_parts = ws.csq_parts;
    OP(SPTS_OP_OPROJ, 2.0 * Ad * Dd * HD, (Ad * HD + 2.0 * Ad * Dd + Dd * HD) * esd, launch_tc_gemm(ctx, TC_RESID, a));
  }
  for (int b = 0; b < n_seq; ++b) caches[b].len = m_attn[b];      // only once everything is enqueued
  return SPTS_OK;
}

spts_status check_ctx(const spts_ctx* ctx) { return ctx == nullptr ? SPTS_ERR_INVALID_ARG : SPTS_OK; }

}  // namespace

extern "C" {

size_t spts_workspace_bytes(const spts_model_desc* desc, int max_seq) {
  if (desc == nullptr || max_seq < 1 || !shape_ok(*desc)) return 0;
  return carve(*desc, max_seq, nullptr, nullptr);
}

spts_status spts_create(const spts_model_desc* desc, int max_seq, void* workspace, size_t workspace_bytes,
                        void* cuda_stream, spts_ctx** out) {
  if (desc == nullptr || out == nullptr || workspace == nullptr || max_seq < 1) return SPTS_ERR_INVALID_ARG;
  if (!shape_ok(*desc)) return SPTS_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return SPTS_ERR_INVALID_ARG;
  if (carve(*desc, max_seq, nullptr, nullptr) > workspace_bytes) return SPTS_ERR_WORKSPACE;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SPTS_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return SPTS_ERR_CUDA;
  if (desc->dtype == SPTS_BF16 && prop.major != 10) return SPTS_ERR_UNSUPPORTED;   // sm_100a only
  spts_ctx* ctx = new (std::nothrow) spts_ctx;
  if (ctx == nullptr) return SPTS_ERR_INVALID_ARG;
  ctx->desc = *desc;
  ctx->max_seq = max_seq;
  ctx->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  ctx->launches = 0;
  ctx->sm_count = prop.multiProcessorCount;
  ctx->encode_tiled = nullptr;
  ctx->ffn_score_pap_only = false;
  ctx->rstd_rows = nullptr;
  ctx->rope_trust = false;
  ctx->rope_pos = nullptr;
  ctx->rope_n = 0;
  ctx->pap_window = 1;
  ctx->debug_checks = false;
  ctx->prof = new (std::nothrow) Profiler;
  ctx->ws_base = reinterpret_cast<char*>(workspace);
  carve(*desc, max_seq, workspace, &ctx->ws, &ctx->guard_offsets);
  for (size_t off : ctx->guard_offsets)
    if (cudaMemsetAsync(ctx->ws_base + off, GUARD_PATTERN, GUARD_BYTES, ctx->stream) != cudaSuccess) {
      spts_destroy(ctx);
      return SPTS_ERR_CUDA;
    }
  ctx->reference_kernels = (desc->dtype == SPTS_FP32) || !tc_shape_ok(*desc);
  if (!ctx->reference_kernels) {
    spts_status s = tc_init(ctx);
    if (s != SPTS_OK) { spts_destroy(ctx); return s; }
  }
  if (cudaMemsetAsync(ctx->ws.status, 0, 64 * sizeof(int), ctx->stream) != cudaSuccess) { spts_destroy(ctx); return SPTS_ERR_CUDA; }
  if (cudaMemsetAsync(ctx->ws.topk_scratch, 0, TOPK_SCRATCH_WORDS * sizeof(uint32_t), ctx->stream) != cudaSuccess) {
    spts_destroy(ctx);
    return SPTS_ERR_CUDA;
  }
  *out = ctx;
  return SPTS_OK;
}

void spts_destroy(spts_ctx* ctx) {
  if (ctx == nullptr) return;
  if (Profiler* p = prof_of(ctx)) {
    for (cudaEvent_t e : p->pool) cudaEventDestroy(e);
    delete p;
  }
  delete ctx;
}

spts_status spts_profile_begin(spts_ctx* ctx, int op) {
  TRY(check_ctx(ctx));
  Profiler* p = prof_of(ctx);
  if (p == nullptr || op < -1 || op >= SPTS_OP_COUNT) return SPTS_ERR_INVALID_ARG;
  p->filter = op;
  p->recs.clear();
  p->used = 0;
  return SPTS_OK;
}

spts_status spts_profile_end(spts_ctx* ctx, float* ms, int64_t* calls, double* flops, double* bytes) {
  TRY(check_ctx(ctx));
  Profiler* p = prof_of(ctx);
  if (p == nullptr || ms == nullptr || calls == nullptr || flops == nullptr || bytes == nullptr) return SPTS_ERR_INVALID_ARG;
  p->filter = 0;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return SPTS_ERR_CUDA;
  for (int i = 0; i < SPTS_OP_COUNT; ++i) { ms[i] = 0.f; calls[i] = 0; flops[i] = 0.0; bytes[i] = 0.0; }
  for (const ProfRecord& r : p->recs) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, r.a, r.b) != cudaSuccess) return SPTS_ERR_CUDA;
    ms[r.tag] += t; calls[r.tag] += 1; flops[r.tag] += r.flops; bytes[r.tag] += r.bytes;
  }
  p->recs.clear();
  p->used = 0;
  return SPTS_OK;
}

spts_status spts_set_option(spts_ctx* ctx, uint32_t option, int value) {
  TRY(check_ctx(ctx));
  if (option == SPTS_REFERENCE_KERNELS) {
    if (ctx->desc.dtype == SPTS_FP32 || !tc_shape_ok(ctx->desc)) return value ? SPTS_OK : SPTS_ERR_UNSUPPORTED;
    if (!value && ctx->encode_tiled == nullptr) TRY(tc_init(ctx));
    ctx->reference_kernels = value != 0;
    return SPTS_OK;
  }
  if (option == SPTS_PAP_WINDOW) {
    if (value < 1 || value > PAP_MAX_WINDOW) return SPTS_ERR_INVALID_ARG;
    ctx->pap_window = value;
    return SPTS_OK;
  }
  if (option == SPTS_DEBUG_CHECKS) {
    ctx->debug_checks = value != 0;
    return SPTS_OK;
  }
  if (option == SPTS_FFN_SCORE_PAP_ONLY) {
    ctx->ffn_score_pap_only = value != 0;
    return SPTS_OK;
  }
  return SPTS_ERR_INVALID_ARG;
}

spts_status spts_last_device_status(spts_ctx* ctx) {
  TRY(check_ctx(ctx));
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return SPTS_ERR_CUDA;
  int st = 0;
  if (cudaMemcpy(&st, ctx->ws.status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return SPTS_ERR_CUDA;
  if (st != 0 && cudaMemset(ctx->ws.status, 0, sizeof(int)) != cudaSuccess) return SPTS_ERR_CUDA;
  return (spts_status)st;
}

int64_t spts_launch_count(const spts_ctx* ctx) { return ctx ? ctx->launches : 0; }

spts_status spts_check_guards(spts_ctx* ctx, int32_t* n_corrupt) {
  TRY(check_ctx(ctx));
  if (n_corrupt == nullptr) return SPTS_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return SPTS_ERR_CUDA;
  unsigned char band[GUARD_BYTES];
  int bad = 0;
  for (size_t off : ctx->guard_offsets) {
    if (cudaMemcpy(band, ctx->ws_base + off, GUARD_BYTES, cudaMemcpyDeviceToHost) != cudaSuccess) return SPTS_ERR_CUDA;
    bool intact = true;
    for (int i = 0; i < GUARD_BYTES; ++i) intact = intact && band[i] == GUARD_PATTERN;
    bad += intact ? 0 : 1;
  }
  *n_corrupt = bad;
  return SPTS_OK;
}

spts_status spts_debug_check_index_list(spts_ctx* ctx, const int32_t* idx, int n, int N) {
  TRY(check_ctx(ctx));
  if (idx == nullptr || n < 1 || N < 1) return SPTS_ERR_INVALID_ARG;
  return launch_check_index_list(ctx, idx, n, N);
}

spts_status spts_selftest_wait_timeout(spts_ctx* ctx, uint32_t limit_us) {
  TRY(check_ctx(ctx));
  if (limit_us < 1 || limit_us > 100000) return SPTS_ERR_INVALID_ARG;
  return launch_wait_selftest(ctx, limit_us);
}

spts_status spts_fold_norm_gain(spts_ctx* ctx, void* W, const float* g, int out_features, int in_features) {
  TRY(check_ctx(ctx));
  if (W == nullptr || g == nullptr || out_features < 1 || in_features < 1) return SPTS_ERR_INVALID_ARG;
  return launch_fold_gain(ctx, W, g, out_features, in_features);
}

size_t spts_prepared_bytes(const spts_model_desc* desc) {
  if (desc == nullptr || !shape_ok(*desc)) return 0;
  return prepared_layout(*desc).total;
}

spts_status spts_prepare_layer(spts_ctx* ctx, const spts_layer_weights* w, void* prepared, size_t prepared_bytes) {
  TRY(check_ctx(ctx));
  if (w == nullptr || prepared == nullptr || w->ug == nullptr || w->uu == nullptr || w->vg == nullptr ||
      w->vu == nullptr || w->ud == nullptr)
    return SPTS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(prepared) & 255) != 0) return SPTS_ERR_INVALID_ARG;
  const PreparedLayout pl = prepared_layout(ctx->desc);
  if (prepared_bytes < pl.total) return SPTS_ERR_WORKSPACE;
  char* base = (char*)prepared;
  return pack_proxy(ctx, w, base + pl.ugu, base + pl.vgu, base + pl.g2);
}

spts_status spts_pap_score(spts_ctx* ctx, const spts_layer_weights* w, const void* X, const int32_t* pos, int N,
                           void* K_out, float* S_mha_out) {
  TRY(check_ctx(ctx));
  if (w == nullptr || X == nullptr || pos == nullptr || S_mha_out == nullptr) return SPTS_ERR_INVALID_ARG;
  if (N < 1 || N > ctx->max_seq) return SPTS_ERR_SHAPE;
  if (!aligned16(X) || !aligned16(K_out) || !aligned16(w->wk) || !aligned16(w->wq)) return SPTS_ERR_INVALID_ARG;
  return pap_pipeline(ctx, w, X, pos, N, K_out ? K_out : ctx->ws.k_all, true, S_mha_out);
}

spts_status spts_ltp_score(spts_ctx* ctx, const spts_layer_weights* w, const void* X, const float* S_mha, int N,
                           float* C_out, float* S_ffn_out) {
  TRY(check_ctx(ctx));
  if (w == nullptr || X == nullptr || S_mha == nullptr || S_ffn_out == nullptr) return SPTS_ERR_INVALID_ARG;
  if (N < 1 || N > ctx->max_seq) return SPTS_ERR_SHAPE;
  if (!aligned16(X)) return SPTS_ERR_INVALID_ARG;
  TRY(launch_rstd(ctx, X, N, ctx->ws.rstd));
  return ltp_pipeline(ctx, w, X, S_mha, N, C_out, S_ffn_out);
}

spts_status spts_topk_select(spts_ctx* ctx, const float* scores, int N, int k, uint32_t flags, int32_t* idx_out) {
  TRY(check_ctx(ctx));
  if (scores == nullptr || idx_out == nullptr) return SPTS_ERR_INVALID_ARG;
  if (N < 1 || k < 1 || k > N) return SPTS_ERR_INVALID_ARG;
  TRY(launch_topk(ctx, scores, N, k, flags, idx_out, ctx->ws.topk_scratch));
  if (ctx->debug_checks) TRY(launch_check_index_list(ctx, idx_out, k, N));
  return SPTS_OK;
}

spts_status spts_layer_prefill_skip(spts_ctx* ctx, const spts_layer_weights* w, void* X, const int32_t* pos, int N,
                                    int m_attn, int m_ffn, uint32_t flags, spts_kv_layer* cache, float* S_mha_out,
                                    int32_t* idx_attn_out, int32_t* idx_ffn_out) {
  TRY(check_ctx(ctx));
  if (w == nullptr || X == nullptr || pos == nullptr || cache == nullptr) return SPTS_ERR_INVALID_ARG;
  if (cache->k == nullptr || cache->v == nullptr || cache->pos == nullptr) return SPTS_ERR_INVALID_ARG;
  if (N < 1 || N > ctx->max_seq) return SPTS_ERR_SHAPE;
  if (m_attn < 1 || m_attn > N || m_ffn < 1 || m_ffn > N) return SPTS_ERR_INVALID_ARG;
  if (cache->capacity < m_attn) return SPTS_ERR_WORKSPACE;
  if (!aligned16(X) || !aligned16(cache->k) || !aligned16(cache->v)) return SPTS_ERR_INVALID_ARG;
  const auto& d = ctx->desc;
  Workspace& ws = ctx->ws;
  const bool sel_f = m_ffn < N;
  float* S = S_mha_out ? S_mha_out : ws.s_mha;
  TRY(attention_block(ctx, w, X, pos, N, m_attn, sel_f || S_mha_out != nullptr, flags, cache, S, idx_attn_out));

  // ---- LTP + reduced FFN on the updated residual
  // ws.rstd still holds the statistics of the layer's input (the probe computed them for every row); only the rows
  // the attention block updated have changed
  if (m_attn < N) {
    const int32_t* ia = idx_attn_out ? idx_attn_out : ws.idx_a;
    OP(SPTS_OP_PREP, 0.0, (double)m_attn * d.hidden * (double)elt_size(d) + 8.0 * m_attn,
       launch_rstd_rows(ctx, X, ia, m_attn, ws.rstd));
  } else {
    OP(SPTS_OP_PREP, 0.0, (double)N * d.hidden * (double)elt_size(d) + 4.0 * N, launch_rstd(ctx, X, N, ws.rstd));
  }
  const int32_t* idx_f = nullptr;
  if (sel_f) {
    int32_t* jf = idx_ffn_out ? idx_ffn_out : ws.idx_f;
    const float* s_ffn = S;                            // Table 4's baseline criterion: the probe's score as it is
    if (!ctx->ffn_score_pap_only) {
      TRY(ltp_pipeline(ctx, w, X, S, N, nullptr, ws.s_ffn));
      s_ffn = ws.s_ffn;
    }
    OP(SPTS_OP_TOPK, 0.0, 4.0 * N + 4.0 * m_ffn, launch_topk(ctx, s_ffn, N, m_ffn, flags, jf, ws.topk_scratch));
    if (ctx->debug_checks) TRY(launch_check_index_list(ctx, jf, m_ffn, N));
    idx_f = jf;
  } else if (idx_ffn_out) {
    TRY(launch_topk(ctx, S, N, N, flags, idx_ffn_out, ws.topk_scratch));
  }
  return ffn_gemms(ctx, w, X, N, idx_f, m_ffn);
}

spts_status spts_reduced_attention(spts_ctx* ctx, const void* Q, const void* K, const void* V, int m, void* O_out) {
  TRY(check_ctx(ctx));
  if (Q == nullptr || K == nullptr || V == nullptr || O_out == nullptr) return SPTS_ERR_INVALID_ARG;
  if (m < 1 || m > ctx->max_seq) return SPTS_ERR_SHAPE;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O_out)) return SPTS_ERR_INVALID_ARG;
  const auto& d = ctx->desc;
  const double Ma = (double)m, HD = (double)d.n_q_heads * d.head_dim, KD = (double)d.n_kv_heads * d.head_dim;
  // the tensor-core kernel reads V through its transposed copy (made outside the timed operation)
  const int ldvt = (int)align_up((size_t)m, 128);
  if (use_tc(ctx)) TRY(launch_transpose_bf16(ctx, V, m, d.n_kv_heads * d.head_dim, ctx->ws.v_t, ldvt));
  ProfScope ps(ctx, SPTS_OP_ATTN, 2.0 * HD * Ma * (Ma + 1.0), (2.0 * Ma * HD + 2.0 * Ma * KD) * (double)elt_size(d));
  if (!use_tc(ctx)) return launch_ref_attention(ctx, Q, K, V, m, O_out);
  return launch_tc_attention(ctx, (const bf16*)Q, (const bf16*)K, (const bf16*)V, (const bf16*)ctx->ws.v_t, ldvt, m,
                             (bf16*)O_out);
}

spts_status spts_layer_prefill_skip_batch(spts_ctx* ctx, const spts_layer_weights* w, void* X, const int32_t* pos,
                                          int n_seq, const int32_t* seq_start, const int32_t* m_attn,
                                          const int32_t* m_ffn, uint32_t flags, spts_kv_layer* caches,
                                          float* S_mha_out, int32_t* idx_attn_out, int32_t* idx_ffn_out) {
  TRY(check_ctx(ctx));
  if (w == nullptr || X == nullptr || pos == nullptr || caches == nullptr || seq_start == nullptr ||
      m_attn == nullptr || m_ffn == nullptr)
    return SPTS_ERR_INVALID_ARG;
  if (n_seq < 1 || seq_start[0] != 0) return SPTS_ERR_INVALID_ARG;
  const int total = seq_start[n_seq];
  if (total < 1 || total > ctx->max_seq) return SPTS_ERR_SHAPE;
  if (!aligned16(X)) return SPTS_ERR_INVALID_ARG;
  bool any_sel_f = false;
  for (int b = 0; b < n_seq; ++b) {
    const int Nb = seq_start[b + 1] - seq_start[b];
    if (Nb < 1) return SPTS_ERR_INVALID_ARG;
    if (m_attn[b] < 1 || m_attn[b] > Nb || m_ffn[b] < 1 || m_ffn[b] > Nb) return SPTS_ERR_INVALID_ARG;
    const spts_kv_layer& c = caches[b];
    if (c.k == nullptr || c.v == nullptr || c.pos == nullptr) return SPTS_ERR_INVALID_ARG;
    if (c.capacity < m_attn[b]) return SPTS_ERR_WORKSPACE;
    if (!aligned16(c.k) || !aligned16(c.v)) return SPTS_ERR_INVALID_ARG;
    any_sel_f = any_sel_f || m_ffn[b] < Nb;
  }
  const auto& d = ctx->desc;
  Workspace& ws = ctx->ws;
  const size_t row_bytes = (size_t)d.hidden * elt_size(d);
  float* S = S_mha_out ? S_mha_out : ws.s_mha;
  int max_len = 0;
  for (int b = 0; b < n_seq; ++b) max_len = seq_start[b + 1] - seq_start[b] > max_len ? seq_start[b + 1] - seq_start[b] : max_len;
  const bool one_launch_per_step = use_tc(ctx) && n_seq <= BATCH_MAX_SEQ && max_len <= TOPK_SEG_MAX && ctx->pap_window < 2 &&
                                   // K^ is packed in the FFN intermediate's buffer: it has to fit there
                                   (size_t)total * d.n_kv_heads * d.head_dim <=
                                       std::min(align_up((size_t)ctx->max_seq, 128), (size_t)FFN_CHUNK_ROWS) * (size_t)d.ffn_dim;
  if (one_launch_per_step) {
    TRY(batch_attention_blocks(ctx, w, X, pos, n_seq, seq_start, m_attn, flags, caches, S, idx_attn_out));
    OP(SPTS_OP_PREP, 0.0, (double)total * (double)row_bytes + 4.0 * total, launch_rstd(ctx, X, total, ws.rstd));
    const float* s_sel = S;
    if (any_sel_f && !ctx->ffn_score_pap_only) {
      TRY(ltp_pipeline(ctx, w, X, S, total, nullptr, ws.s_ffn));
      s_sel = ws.s_ffn;
    }
    // TopK of Eq. 15 per sequence in one launch; the tables of budgets and offsets follow the attention block's
    std::vector<int32_t> tab((size_t)2 * (n_seq + 1), 0);
    int F = 0;
    for (int b = 0; b < n_seq; ++b) { tab[b] = m_ffn[b]; tab[n_seq + 1 + b] = F; F += m_ffn[b]; }
    tab[2 * n_seq + 1] = F;
    int32_t* d_mf = ws.batch_i32 + 4 * (n_seq + 1);
    int32_t* d_foff = d_mf + (n_seq + 1);
    if (any_sel_f || idx_ffn_out != nullptr) {
      if (cudaMemcpyAsync(d_mf, tab.data(), tab.size() * sizeof(int32_t), cudaMemcpyHostToDevice, ctx->stream) != cudaSuccess)
        return SPTS_ERR_CUDA;
      OP(SPTS_OP_TOPK, 0.0, 4.0 * total + 4.0 * F,
         launch_topk_segmented(ctx, s_sel, ws.batch_i32, d_mf, d_foff, n_seq, max_len, flags, idx_ffn_out, ws.idx_f));
      if (ctx->debug_checks && any_sel_f) TRY(launch_check_index_list(ctx, ws.idx_f, F, total));
    }
    return ffn_gemms(ctx, w, X, total, any_sel_f ? ws.idx_f : nullptr, F);
  }
  // ---- attention blocks, one sequence after the other: the probe's softmax, the selection and the causal mask
  //      are per sequence.  The rotary table is rebuilt for every slice.
  int off_a = 0;
  for (int b = 0; b < n_seq; ++b) {
    const int s0 = seq_start[b], Nb = seq_start[b + 1] - s0;
    ctx->rope_trust = false;
    TRY(attention_block(ctx, w, (char*)X + (size_t)s0 * row_bytes, pos + s0, Nb, m_attn[b],
                        m_ffn[b] < Nb || S_mha_out != nullptr, flags, &caches[b], S + s0,
                        idx_attn_out ? idx_attn_out + off_a : nullptr));
    off_a += m_attn[b];
  }
  // ---- FFN block over the packed rows: one norm pass, one proxy chain, one gathered FFN for all sequences
  OP(SPTS_OP_PREP, 0.0, (double)total * (double)row_bytes + 4.0 * total, launch_rstd(ctx, X, total, ws.rstd));
  const float* s_ffn = S;
  if (any_sel_f && !ctx->ffn_score_pap_only) {
    TRY(ltp_pipeline(ctx, w, X, S, total, nullptr, ws.s_ffn));
    s_ffn = ws.s_ffn;
  }
  int off_f = 0;
  for (int b = 0; b < n_seq; ++b) {
    const int s0 = seq_start[b], Nb = seq_start[b + 1] - s0, mf = m_ffn[b];
    int32_t* local = idx_ffn_out ? idx_ffn_out + off_f : ws.idx_p;
    if (mf < Nb) {
      OP(SPTS_OP_TOPK, 0.0, 4.0 * Nb + 4.0 * mf, launch_topk(ctx, s_ffn + s0, Nb, mf, flags, local, ws.topk_scratch));
      if (any_sel_f) TRY(launch_offset_i32(ctx, local, mf, s0, ws.idx_f + off_f));
    } else {
      if (idx_ffn_out) TRY(launch_iota_from(ctx, local, Nb, 0));
      if (any_sel_f) TRY(launch_iota_from(ctx, ws.idx_f + off_f, Nb, s0));
    }
    off_f += mf;
  }
  if (ctx->debug_checks && any_sel_f) TRY(launch_check_index_list(ctx, ws.idx_f, off_f, total));
  return ffn_gemms(ctx, w, X, total, any_sel_f ? ws.idx_f : nullptr, off_f);
}

spts_status spts_msdp_compact(spts_ctx* ctx, const void* X_in, const int32_t* pos_in, const int32_t* orig_in,
                              const float* S_mha, int N, int n_next, uint32_t flags, void* X_out, int32_t* pos_out,
                              int32_t* orig_out, int32_t* idx_out) {
  TRY(check_ctx(ctx));
  if (X_in == nullptr || pos_in == nullptr || orig_in == nullptr || S_mha == nullptr || X_out == nullptr ||
      pos_out == nullptr || orig_out == nullptr)
    return SPTS_ERR_INVALID_ARG;
  if (X_in == X_out || pos_in == pos_out || orig_in == orig_out) return SPTS_ERR_INVALID_ARG;
  if (N < 1 || N > ctx->max_seq || n_next < 1) return SPTS_ERR_SHAPE;
  if (n_next > N) n_next = N;
  if (!aligned16(X_in) || !aligned16(X_out)) return SPTS_ERR_INVALID_ARG;
  int32_t* idx = idx_out ? idx_out : ctx->ws.idx_p;
  OP(SPTS_OP_TOPK, 0.0, 4.0 * N + 4.0 * n_next, launch_topk(ctx, S_mha, N, n_next, flags, idx, ctx->ws.topk_scratch));
  if (ctx->debug_checks) TRY(launch_check_index_list(ctx, idx, n_next, N));
  ProfScope ps_c(ctx, SPTS_OP_COMPACT, 0.0, 2.0 * n_next * (double)ctx->desc.hidden * (double)elt_size(ctx->desc) + 28.0 * n_next);
  TRY(launch_gather_rows(ctx, X_in, idx, n_next, (int)(ctx->desc.hidden * elt_size(ctx->desc)), X_out));
  TRY(launch_gather_i32(ctx, pos_in, idx, n_next, pos_out));
  TRY(launch_gather_i32(ctx, orig_in, idx, n_next, orig_out));
  return SPTS_OK;
}

spts_status spts_msdp_plan(int n_layers, int n_prompt, int skip_from, const spts_msdp_stage* stages, int n_stages,
                           spts_layer_plan* plan_out, int32_t* n_final, int64_t* kv_token_layers) {
  if (stages == nullptr || plan_out == nullptr || n_layers < 1 || n_prompt < 1 || n_stages < 1) return SPTS_ERR_INVALID_ARG;
  for (int s = 1; s < n_stages; ++s)
    if (stages[s].last_layer <= stages[s - 1].last_layer) return SPTS_ERR_INVALID_ARG;
  int cur = n_prompt, s = 0;
  int64_t kv = 0;
  for (int l = 0; l < n_layers; ++l) {
    while (s + 1 < n_stages && stages[s].last_layer < l) ++s;
    const spts_msdp_stage& st = stages[s];
    spts_layer_plan p;
    const bool skip = l >= skip_from;
    p.m_attn = (skip && st.m_attn_fixed > 0 && st.m_attn_fixed < cur) ? st.m_attn_fixed : cur;   // M^l = min(|T^l|, M_fixed)
    p.m_ffn = (skip && st.m_ffn_fixed > 0 && st.m_ffn_fixed < cur) ? st.m_ffn_fixed : cur;
    p.prune_to = (l == st.last_layer && st.n_next > 0 && st.n_next < cur) ? st.n_next : 0;       // |T^{l+1}| of Eq. 16
    plan_out[l] = p;
    kv += p.m_attn;
    if (p.prune_to) cur = p.prune_to;
  }
  if (n_final) *n_final = cur;
  if (kv_token_layers) *kv_token_layers = kv;
  return SPTS_OK;
}

namespace {
constexpr int PROXY_SWEEPS = 14;
struct ProxyScratch {
  float* rstd; float* zt; int ld; float* importance; int32_t* channels; float* A; float* V; float* sigma;
  int32_t* order; unsigned int* offdiag;
};
size_t carve_proxy(const spts_model_desc& d, int n_cal, void* base, ProxyScratch* out) {
  Carver c{reinterpret_cast<char*>(base), 0, nullptr};
  ProxyScratch p;
  p.ld = (int)align_up((size_t)n_cal, 32);
  p.rstd = c.take<float>((size_t)n_cal);
  p.zt = c.take<float>((size_t)d.ffn_dim * p.ld);
  p.importance = c.take<float>((size_t)d.ffn_dim);
  p.channels = c.take<int32_t>((size_t)d.ltp_dlow);
  p.A = c.take<float>((size_t)d.ltp_dlow * d.hidden);
  p.V = c.take<float>((size_t)d.ltp_dlow * d.ltp_dlow);
  p.sigma = c.take<float>((size_t)d.ltp_dlow);
  p.order = c.take<int32_t>((size_t)d.ltp_dlow);
  p.offdiag = c.take<unsigned int>(64);
  if (out) *out = p;
  return align_up(c.off, 256);
}
}  // namespace

size_t spts_proxy_scratch_bytes(const spts_model_desc* desc, int n_cal) {
  if (desc == nullptr || n_cal < 1 || !shape_ok(*desc)) return 0;
  return carve_proxy(*desc, n_cal, nullptr, nullptr);
}

spts_status spts_proxy_build(spts_ctx* ctx, const spts_layer_weights* w, const void* calib, int n_cal, double rho,
                             void* scratch, size_t scratch_bytes, float* importance_out, int32_t* channels_out,
                             void* ug, void* vg, void* uu, void* vu, void* vd, void* ud, float* sigma_out) {
  TRY(check_ctx(ctx));
  if (w == nullptr || calib == nullptr || scratch == nullptr || ug == nullptr || vg == nullptr || uu == nullptr ||
      vu == nullptr || vd == nullptr || ud == nullptr || w->w_gate == nullptr || w->w_up == nullptr ||
      w->w_down == nullptr)
    return SPTS_ERR_INVALID_ARG;
  const auto& d = ctx->desc;
  if (n_cal < 1 || !(rho > 0.0) || rho > 1.0) return SPTS_ERR_INVALID_ARG;
  if (d.ltp_dlow > d.ffn_dim || d.ltp_dlow % 2 != 0 || d.ltp_rank > d.ltp_dlow || d.ltp_rank > d.hidden) return SPTS_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(scratch) & 255) != 0 || !aligned16(calib)) return SPTS_ERR_INVALID_ARG;
  if (carve_proxy(d, n_cal, nullptr, nullptr) > scratch_bytes) return SPTS_ERR_WORKSPACE;
  ProxyScratch ps;
  carve_proxy(d, n_cal, scratch, &ps);
  float* imp = importance_out ? importance_out : ps.importance;
  int32_t* ch = channels_out ? channels_out : ps.channels;
  // saliency z(x) = |silu(x W_gate) * (x W_up)| of every calibration token, one row per channel
  TRY(launch_rstd(ctx, calib, n_cal, ps.rstd));
  Gemm g;
  memset(&g, 0, sizeof(g));
  g.A = calib; g.lda = d.hidden; g.a_rows = n_cal; g.W = w->w_gate; g.W2 = w->w_up; g.M = n_cal; g.Nout = d.ffn_dim;
  g.K = d.hidden; g.rowscale = ps.rstd; g.sal_t = ps.zt; g.ld_sal = ps.ld;
  TRY(run_gemm(ctx, REF_SWIGLU, g));
  // channel importance: mean of the top rho-fraction per channel, then the D_low most important channels
  int k = (int)floor(rho * (double)n_cal);
  if (k < 1) k = 1;
  TRY(launch_proxy_importance(ctx, ps.zt, ps.ld, n_cal, k, d.ffn_dim, imp));
  TRY(launch_topk(ctx, imp, d.ffn_dim, d.ltp_dlow, 0u, ch, ctx->ws.topk_scratch));
  // W' = W[:, C] ~ U V for the three projections
  const int n = d.ltp_dlow;
  TRY(launch_proxy_factor(ctx, w->w_gate, ch, 0, PROXY_SWEEPS, ps.A, ps.V, ps.sigma, ps.order, ps.offdiag, d.ltp_rank,
                          ug, vg, sigma_out ? sigma_out : nullptr));
  TRY(launch_proxy_factor(ctx, w->w_up, ch, 0, PROXY_SWEEPS, ps.A, ps.V, ps.sigma, ps.order, ps.offdiag + 16, d.ltp_rank,
                          uu, vu, sigma_out ? sigma_out + n : nullptr));
  TRY(launch_proxy_factor(ctx, w->w_down, ch, 1, PROXY_SWEEPS, ps.A, ps.V, ps.sigma, ps.order, ps.offdiag + 32, d.ltp_rank,
                          ud, vd, sigma_out ? sigma_out + 2 * n : nullptr));
  return SPTS_OK;
}

spts_status spts_first_token(spts_ctx* ctx, const void* x_row, const void* lm_head, float* logits_out,
                             int32_t* token_out) {
  TRY(check_ctx(ctx));
  if (x_row == nullptr || lm_head == nullptr || ctx->desc.vocab < 1) return SPTS_ERR_INVALID_ARG;
  if (!aligned16(x_row) || !aligned16(lm_head)) return SPTS_ERR_INVALID_ARG;
  ProfScope ps_h(ctx, SPTS_OP_HEAD, 2.0 * ctx->desc.vocab * (double)ctx->desc.hidden,
                 ctx->desc.vocab * ((double)ctx->desc.hidden * (double)elt_size(ctx->desc) + 8.0));
  return launch_head(ctx, x_row, lm_head, logits_out ? logits_out : ctx->ws.logits_v, token_out);
}

spts_status spts_prefill(spts_ctx* ctx, const spts_model_weights* mw, const spts_layer_plan* plan, void* X,
                         int32_t* pos, int32_t* orig, void* X_alt, int32_t* pos_alt, int32_t* orig_alt, int N,
                         uint32_t flags, spts_kv_layer* caches, int32_t* n_final, int32_t* final_in_alt,
                         int32_t* token_out) {
  TRY(check_ctx(ctx));
  if (mw == nullptr || mw->layers == nullptr || plan == nullptr || X == nullptr || pos == nullptr || orig == nullptr ||
      caches == nullptr)
    return SPTS_ERR_INVALID_ARG;
  if (N < 1 || N > ctx->max_seq) return SPTS_ERR_SHAPE;
  const auto& d = ctx->desc;
  // the caller's pos buffers are only written by this call's own compactions while it runs, so a rotary table
  // stays valid until the buffers swap
  struct RopeTrust {
    spts_ctx* c;
    explicit RopeTrust(spts_ctx* cc) : c(cc) { c->rope_trust = true; c->rope_pos = nullptr; c->rstd_rows = nullptr; }
    ~RopeTrust() { c->rope_trust = false; c->rope_pos = nullptr; c->rstd_rows = nullptr; }
  } rope_guard(ctx);
  void* xc = X; int32_t* pc = pos; int32_t* oc = orig;
  void* xa = X_alt; int32_t* pa = pos_alt; int32_t* oa = orig_alt;
  int cur = N, in_alt = 0;
  for (int l = 0; l < d.n_layers; ++l) {
    const spts_layer_plan& p = plan[l];
    if (p.m_attn < 1 || p.m_attn > cur || p.m_ffn < 1 || p.m_ffn > cur) return SPTS_ERR_INVALID_ARG;
    const bool prune = p.prune_to > 0 && p.prune_to < cur;
    if (prune && (xa == nullptr || pa == nullptr || oa == nullptr)) return SPTS_ERR_INVALID_ARG;
    TRY(spts_layer_prefill_skip(ctx, &mw->layers[l], xc, pc, cur, p.m_attn, p.m_ffn, flags, &caches[l],
                                prune ? ctx->ws.s_mha : nullptr, nullptr, nullptr));
    // The layer left ws.rstd current for its post-attention residual; its FFN block then changed the rows in
    // ws.idx_f only.  Without a compaction the next layer's first norm pass can be limited to those rows.
    ctx->rstd_rows = nullptr;
    if (!prune && p.m_ffn < cur) {
      ctx->rstd_rows = ctx->ws.idx_f; ctx->rstd_nrows = p.m_ffn; ctx->rstd_x = xc; ctx->rstd_n = cur;
    }
    if (prune) {
      TRY(spts_msdp_compact(ctx, xc, pc, oc, ctx->ws.s_mha, cur, p.prune_to, flags, xa, pa, oa, nullptr));
      void* tx = xc; xc = xa; xa = tx;
      int32_t* tp = pc; pc = pa; pa = tp;
      int32_t* to = oc; oc = oa; oa = to;
      cur = p.prune_to;
      in_alt ^= 1;
    }
  }
  if (n_final) *n_final = cur;
  if (final_in_alt) *final_in_alt = in_alt;
  if (token_out != nullptr) {
    if (mw->lm_head == nullptr) return SPTS_ERR_INVALID_ARG;
    const char* last = (const char*)xc + (size_t)(cur - 1) * d.hidden * elt_size(d);
    TRY(spts_first_token(ctx, last, mw->lm_head, nullptr, token_out));
  }
  return SPTS_OK;
}

spts_status spts_decode_step(spts_ctx* ctx, const spts_model_weights* mw, spts_kv_layer* caches, const void* x_in,
                             int32_t token_in, int32_t pos, void* x_out, float* logits_out, int32_t* token_out) {
  TRY(check_ctx(ctx));
  if (mw == nullptr || mw->layers == nullptr || caches == nullptr) return SPTS_ERR_INVALID_ARG;
  const auto& d = ctx->desc;
  const size_t es = elt_size(d);
  const void* x = x_in;
  if (x == nullptr) {
    if (mw->embed == nullptr || token_in < 0 || token_in >= d.vocab) return SPTS_ERR_INVALID_ARG;
    x = (const char*)mw->embed + (size_t)token_in * d.hidden * es;
  }
  for (int l = 0; l < d.n_layers; ++l)
    if (caches[l].len + 1 > caches[l].capacity) return SPTS_ERR_WORKSPACE;
  double kvb = 0.0;
  for (int l = 0; l < d.n_layers; ++l) kvb += 2.0 * (caches[l].len + 1.0) * d.n_kv_heads * d.head_dim * (double)es;
  const double wl = ((2.0 * d.n_q_heads + 2.0 * d.n_kv_heads) * d.head_dim + 3.0 * d.ffn_dim) * (double)d.hidden;
  ProfScope* ps_d = new ProfScope(ctx, SPTS_OP_DECODE, 2.0 * wl * d.n_layers, wl * d.n_layers * (double)es + kvb);
  struct Guard { ProfScope* p; ~Guard() { delete p; } } guard_d{ps_d};
  TRY(launch_decode_load(ctx, x));
  for (int l = 0; l < d.n_layers; ++l) TRY(launch_decode_layer(ctx, &mw->layers[l], &caches[l], pos));
  // the residual is already rounded through the storage type; park it where the head can read it
  void* xo = x_out ? x_out : ctx->ws.xrow;
  TRY(launch_decode_store(ctx, xo));
  // every layer is enqueued: only now do the caches grow on the host side, so a launch error in the middle of a
  // step leaves all lengths as they were
  for (int l = 0; l < d.n_layers; ++l) caches[l].len += 1;
  delete guard_d.p; guard_d.p = nullptr;
  if (logits_out != nullptr || token_out != nullptr) {
    if (mw->lm_head == nullptr) return SPTS_ERR_INVALID_ARG;
    TRY(launch_head(ctx, xo, mw->lm_head, logits_out ? logits_out : ctx->ws.logits_v, token_out));
  }
  return SPTS_OK;
}

}  // extern "C"
