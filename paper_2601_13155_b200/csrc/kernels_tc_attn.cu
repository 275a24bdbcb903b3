// Causal GQA attention among the m active rows (Algorithm 1: O^ <- F_MHA(Q^, K^, V^)) on tcgen05.
// Index lists are ascending, so causality among the selected tokens is a lower triangle in the
// compact row order.
//
// tc_attention_pair_kernel: one CTA = two score tiles of 128 queries that read the same K / V: two
// query heads that share a KV head (even GQA group, grid = (H / 2, ceil(m / 128))), or else two
// consecutive query tiles of one head (grid = (H, ceil(m / 256)); the earlier tile then sits out the
// last key block).  Every K_j / V_j tile staged in shared memory feeds two score tiles, and the
// tensor core always has the other tile's MMAs to run while one tile's softmax is in progress.
// Longest query tiles first.
//   warp 0      TMA producer: both Q tiles and K_0 once, then per key block the pair (V^T_j, K_{j+1})
//               [128 x 128 each] under one barrier
//   warp 1      TMEM owner and single-thread MMA issuer.  TMEM columns: S_0 | S_1 | O_0 | O_1
//               (4 x 128 fp32 columns).  Per key block j and tile t:  O_t += P_t V_j  (A operand P_t
//               read from TMEM, where it overwrites the first 64 columns of S_t; issued piece by
//               piece as the softmax warps deliver it), then S_t = Q_t K_{j+1}^T.
//   warps 2-3   no role (they fill the first warp group, whose registers are handed to the softmax warps)
//   warps 4-7   softmax of tile 0, warps 8-11 softmax of tile 1; one query row per thread, the whole score
//               row in registers: row maximum, p = 2^(s * log2(e)/sqrt(d) - max) with a lazily updated running maximum (O_t
//               is rescaled in TMEM only when the maximum grows by more than 2^8), row sum, P_t
//               written back to TMEM as packed bf16; at the end O_t / l goes to global memory.
#include "spts_common.cuh"
#include "tc_ptx.cuh"

namespace spts {

spts_status tc_gemm_init(spts_ctx* ctx);

namespace {

using namespace ptx;

constexpr int TILE = 128;                    // queries per CTA, keys per block, head dim
constexpr int SLAB_BYTES = TILE * 128;       // [128 rows x 64 bf16] swizzled slab = 16 KiB
constexpr int TILE_BYTES = 2 * SLAB_BYTES;   // 32 KiB
constexpr int KV_STAGES = 2;
constexpr int AT_TMEM_COLS = 512;
constexpr float RESCALE_THRESHOLD = 8.0f;    // log2 units

struct AttnParams {
  int m, H, Hkv;
  int pair_tiles;   // 0 = the CTA's two tiles are two heads of one KV head, 1 = two query tiles of one head
  bf16* O;          // [m, H*128]
  int* status;
  // Packed batch (nullptr: one sequence of m rows starting at row 0).  Entry blockIdx.y = (first row of the sequence in
  // the packed Q / K^ / O buffers, its first column in the packed V^T, its row count, the query tile (or tile pair) of
  // that sequence this CTA takes); longest tiles first.
  const int4* tiles;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Warp group 0: TMA warp, MMA warp, two warps with no role; warp groups 1 and 2: the softmax of tile 0 and of tile 1.
// Registers live per SM sub-partition (16384 each, three warps of this block on every one), so an even split caps a
// thread at 168.  The light warp group hands registers back (setmaxnreg works on whole warp groups, hence the two
// idle warps) and a softmax thread -- which keeps a whole 128-entry score row plus its packed probabilities in
// registers -- gets 224: the same kernel with the softmax squeezed into 168 registers ran 6 % slower.
constexpr int AP_THREADS = 384;
constexpr int REGS_LIGHT = 56, REGS_SOFTMAX = 224;   // 128 * 56 + 256 * 224 = 384 * 168

__device__ __forceinline__ void setmaxnreg_dec_light() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_LIGHT)); }
__device__ __forceinline__ void setmaxnreg_inc_softmax() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_SOFTMAX)); }
constexpr int AP_SMEM = 2 * TILE_BYTES /*Q_0, Q_1*/ + KV_STAGES * TILE_BYTES /*K*/ + KV_STAGES * TILE_BYTES /*V^T*/ +
                        1024 + 256;

constexpr int P_PARTS = 2;                   // pieces (64 keys each) in which a P tile is handed to the MMA warp

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

__global__ void __launch_bounds__(AP_THREADS, 1)
tc_attention_pair_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                         const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = base;                                  // two tiles
  const uint32_t sK = sQ + 2 * TILE_BYTES;
  const uint32_t sV = sK + KV_STAGES * TILE_BYTES;
  const uint32_t bars = sV + KV_STAGES * TILE_BYTES;
  const uint32_t q_full = bars;
  // K and V travel in pairs: stage j & 1 holds V_j and K_{j+1}, the two tiles key block j's MMAs
  // (P_t V_j, then Q_t K_{j+1}^T) read, so one wait and one release per block serve both
  const uint32_t kv_full = bars + 8;         // [2 stages]
  const uint32_t kv_free = bars + 24;        // [2]
  const uint32_t s_full = bars + 40;         // [2 tiles]  S_t of the next key block is complete
  const uint32_t o_full = bars + 56;         // [2 tiles]  last P_t V_j done
  const uint32_t p_full = bars + 72;         // [2 tiles][P_PARTS]  a piece of P_t written by its 128 softmax threads
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + (bars - base) + 128);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Tile t of the CTA is (head_t, query tile qt_t).  Even GQA groups: two heads that share a KV head, same query
  // tile (both tiles see the same key blocks).  Otherwise: two consecutive query tiles of one head; tile 0 then has
  // one key block fewer than tile 1 and sits out the last block.
  int yy = (int)gridDim.y - 1 - (int)blockIdx.y;              // longest tiles first
  int row0 = 0, vcol0 = 0, m_rows = p.m;
  if (p.tiles != nullptr) {
    const int4 e = p.tiles[blockIdx.y];
    row0 = e.x; vcol0 = e.y; m_rows = e.z; yy = e.w;
  }
  const int h0 = p.pair_tiles ? (int)blockIdx.x : 2 * (int)blockIdx.x;
  const int qt0 = p.pair_tiles ? 2 * yy : yy;
  const int dh = p.pair_tiles ? 0 : 1, dq = p.pair_tiles ? 1 : 0;   // head / query-tile step from tile 0 to tile 1
  const int kvh = h0 / (p.H / p.Hkv);
  const int nblk = qt0 + dq + 1;                               // key blocks of the longer tile
  const uint64_t t0 = globaltimer_ns();

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(q_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(kv_full + 8 * s, 1); mbar_init(kv_free + 8 * s, 1);
      mbar_init(s_full + 8 * s, 1); mbar_init(o_full + 8 * s, 1);
      for (int part = 0; part < P_PARTS; ++part) mbar_init(p_full + 8 * (P_PARTS * s + part), 128);
    }
    fence_mbar_init();
    prefetch_tensormap(&tmQ); prefetch_tensormap(&tmK); prefetch_tensormap(&tmV);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32((const void*)tmem_slot), AT_TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // the register hand-over brackets each warp group's whole role: code after a join of the two branches would have to
  // fit the smaller allowance
  if (warp < 4) {
  setmaxnreg_dec_light();
  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(q_full, 3 * TILE_BYTES);               // both Q tiles and K_0 (K_j sits in slot (j + 1) & 1)
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        tma_load_2d(sQ + t * TILE_BYTES, &tmQ, q_full, (h0 + t * dh) * TILE, row0 + (qt0 + t * dq) * TILE);
        tma_load_2d(sQ + t * TILE_BYTES + SLAB_BYTES, &tmQ, q_full, (h0 + t * dh) * TILE + 64, row0 + (qt0 + t * dq) * TILE);
      }
      tma_load_2d(sK + TILE_BYTES, &tmK, q_full, kvh * TILE, row0);
      tma_load_2d(sK + TILE_BYTES + SLAB_BYTES, &tmK, q_full, kvh * TILE + 64, row0);
      bool ok = true;
      for (int j = 0; j < nblk && ok; ++j) {
        const int s = j & 1;
        const bool more = j + 1 < nblk;
        // stage 1 starts occupied (its K slot holds K_0) and is first released after Q_t K_0^T, so its
        // releases run one ahead of stage 0's
        ok = mbar_wait(kv_free + 8 * s, ((uint32_t)(j >> 1) & 1u) ^ (uint32_t)(s ^ 1), abort_flag, t0);
        if (!ok) break;
        mbar_expect_tx(kv_full + 8 * s, more ? 2 * TILE_BYTES : TILE_BYTES);
        tma_load_2d(sV + s * TILE_BYTES, &tmV, kv_full + 8 * s, vcol0 + j * TILE, kvh * TILE);
        tma_load_2d(sV + s * TILE_BYTES + SLAB_BYTES, &tmV, kv_full + 8 * s, vcol0 + j * TILE + 64, kvh * TILE);
        if (more) {
          tma_load_2d(sK + s * TILE_BYTES, &tmK, kv_full + 8 * s, kvh * TILE, row0 + (j + 1) * TILE);
          tma_load_2d(sK + s * TILE_BYTES + SLAB_BYTES, &tmK, kv_full + 8 * s, kvh * TILE + 64, row0 + (j + 1) * TILE);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16(TILE, TILE);
      // S_t = Q_t K_j^T
      auto issue_qk = [&](int t, int j) {
        const uint32_t kb = sK + ((j + 1) & 1) * TILE_BYTES, qb = sQ + t * TILE_BYTES;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t off = (k >> 2) * SLAB_BYTES + (k & 3) * 32;
          mma_bf16(tmem_base + t * TILE, smem_desc_sw128(qb + off), smem_desc_sw128(kb + off), idesc, k > 0 ? 1u : 0u);
        }
      };
      // O_t += P_t V_j for the keys of piece `part`, P_t read from the columns of S_t
      auto issue_pv = [&](int t, int j, int part) {
        const uint32_t vb = sV + (j & 1) * TILE_BYTES;
#pragma unroll
        for (int kk = 0; kk < 8 / P_PARTS; ++kk) {
          const int k = part * (8 / P_PARTS) + kk;
          const uint32_t off = (k >> 2) * SLAB_BYTES + (k & 3) * 32;
          mma_bf16_tmem_a(tmem_base + 2 * TILE + t * TILE, tmem_base + t * TILE + k * 8, smem_desc_sw128(vb + off), idesc,
                          (j > 0 || k > 0) ? 1u : 0u);
        }
      };
      bool ok = mbar_wait(q_full, 0, abort_flag, t0);
      if (ok) {
        tc_fence_after();
        issue_qk(0, 0);
        mma_commit(s_full);
        issue_qk(1, 0);
        mma_commit(s_full + 8);
        mma_commit(kv_free + 8);             // K_0's slot may be refilled (with K_2) once these are done
      }
      for (int j = 0; j < nblk && ok; ++j) {
        const int sv = j & 1;
        ok = mbar_wait(kv_full + 8 * sv, (uint32_t)(j >> 1) & 1u, abort_flag, t0);
        if (!ok) break;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          const int nblk_t = qt0 + t * dq + 1;
          if (j >= nblk_t) continue;                    // the shorter tile has no such key block
          const bool more_t = j + 1 < nblk_t;
          // P_t arrives in P_PARTS pieces (one barrier each), so the first MMAs of P_t V_j run while
          // the softmax warps are still computing the exponentials of the later keys
#pragma unroll
          for (int part = 0; part < P_PARTS; ++part) {
            ok = mbar_wait(p_full + 8 * (P_PARTS * t + part), (uint32_t)j & 1u, abort_flag, t0);
            if (!ok) break;
            tc_fence_after();
            issue_pv(t, j, part);
          }
          if (!ok) break;
          if (more_t) {
            issue_qk(t, j + 1);
            mma_commit(s_full + 8 * t);       // also covers P_t V_j: O_t is quiescent when S_t arrives
          } else {
            mma_commit(o_full + 8 * t);
          }
        }
        if (!ok) break;
        mma_commit(kv_free + 8 * sv);
      }
    }
  }
  } else {
    setmaxnreg_inc_softmax();
    // ------------------------------------------------------------------ softmax / rescale / epilogue
    const int t = (warp - 4) >> 2;                     // tile
    const int qt = qt0 + t * dq, head = h0 + t * dh;
    const int nblk_t = qt + 1;
    const int quarter = warp & 3;                      // TMEM lane quarter this warp may access
    const int row = quarter * 32 + lane;
    const int qi = qt * TILE + row;                    // compact query index
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const uint32_t tSt = tmem_base + t * TILE + lane_off;
    const uint32_t tOt = tmem_base + 2 * TILE + t * TILE + lane_off;
    const float sc = 0.08838834764831845f * 1.4426950408889634f;   // log2(e) / sqrt(128)
    const float2 sc2 = make_float2(sc, sc);
    float m_used = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < nblk_t && ok; ++j) {
      ok = mbar_wait(s_full + 8 * t, (uint32_t)j & 1u, abort_flag, t0);
      if (!ok) break;
      tc_fence_after();
      const bool diag = (j == qt);
      const int key0 = j * TILE;
      // the whole score row into registers: four loads in flight, one wait
      uint32_t r[TILE];
#pragma unroll
      for (int c = 0; c < TILE; c += 32) tmem_ld32(tSt + c, r + c);
      tmem_ld_wait();
      if (diag) {
#pragma unroll
        for (int i = 0; i < TILE; ++i)
          if (key0 + i > qi) r[i] = 0xFF800000u;        // -inf: keys after the query
      }
      // row maximum of the raw scores (four independent chains)
      float bm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int i = 0; i < TILE; i += 8) {
#pragma unroll
        for (int u = 0; u < 4; ++u) bm[u] = max3(bm[u], __uint_as_float(r[i + 2 * u]), __uint_as_float(r[i + 2 * u + 1]));
      }
      const float bmax = fmaxf(fmaxf(bm[0], bm[1]), fmaxf(bm[2], bm[3])) * sc;
      float alpha = 1.0f;      // factor applied to O and l when the running maximum is replaced
      if (bmax > m_used + RESCALE_THRESHOLD || m_used == -INFINITY) {
        alpha = (m_used == -INFINITY) ? 0.0f : ex2(m_used - bmax);
        m_used = bmax;
      }
      // S_t complete means P_t V_{j-1} has completed too, and P_t V_j cannot start before this thread's
      // P arrives: O_t is safe to rescale here
      if (j >= 1 && __any_sync(0xffffffffu, alpha != 1.0f)) {
#pragma unroll 1
        for (int c = 0; c < TILE; c += 32) {
          uint32_t o[32];
          tmem_ld32(tOt + c, o);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
          tmem_st32(tOt + c, o);
        }
      }
      // p = 2^(s * sc - m), row sum, bf16 pairs written over the first half of S_t, handed over in
      // P_PARTS pieces.  The first piece's wait::st also covers the O_t rescale stores above.
      const float2 nm2 = make_float2(-m_used, -m_used);
      float2 ps[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) ps[u] = make_float2(0.f, 0.f);
#pragma unroll
      for (int part = 0; part < P_PARTS; ++part) {
        constexpr int PE = TILE / P_PARTS;             // elements per piece
        uint32_t pk[PE / 2];
#pragma unroll
        for (int i = 0; i < PE; i += 2) {
          const int e0 = part * PE + i;
          const float2 x = __ffma2_rn(make_float2(__uint_as_float(r[e0]), __uint_as_float(r[e0 + 1])), sc2, nm2);
          const float2 e = make_float2(ex2(x.x), ex2(x.y));
          ps[(i >> 1) & 3] = __fadd2_rn(ps[(i >> 1) & 3], e);
          pk[i >> 1] = pack2(e.x, e.y);
        }
#pragma unroll
        for (int c = 0; c < PE / 2; c += 16) tmem_st16(tSt + part * (PE / 2) + c, pk + c);
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(p_full + 8 * (P_PARTS * t + part));
      }
      const float2 ps0 = __fadd2_rn(ps[0], ps[1]), ps1 = __fadd2_rn(ps[2], ps[3]);
      l = l * alpha + ((ps0.x + ps0.y) + (ps1.x + ps1.y));
    }
    // ---- epilogue: O_t / l
    if (ok) ok = mbar_wait(o_full + 8 * t, 0, abort_flag, t0);
    if (ok) {
      tc_fence_after();
      const float inv = 1.0f / l;
      bf16* orow = p.O + ((size_t)(row0 + qi) * p.H + head) * TILE;
#pragma unroll 1
      for (int c = 0; c < TILE; c += 32) {
        uint32_t r[32];
        tmem_ld32(tOt + c, r);
        tmem_ld_wait();
        if (qi < m_rows) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint4 w;
            w.x = pack2(__uint_as_float(r[g * 8 + 0]) * inv, __uint_as_float(r[g * 8 + 1]) * inv);
            w.y = pack2(__uint_as_float(r[g * 8 + 2]) * inv, __uint_as_float(r[g * 8 + 3]) * inv);
            w.z = pack2(__uint_as_float(r[g * 8 + 4]) * inv, __uint_as_float(r[g * 8 + 5]) * inv);
            w.w = pack2(__uint_as_float(r[g * 8 + 6]) * inv, __uint_as_float(r[g * 8 + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + c + g * 8) = w;
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) set_status(p.status, SPTS_ERR_TIMEOUT);
    const uint64_t t1 = globaltimer_ns();
    while (globaltimer_ns() - t1 < 200000ull) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, AT_TMEM_COLS);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool make_map(spts_ctx* ctx, CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint64_t ld) {
  EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstride[1] = {ld * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)TILE};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

spts_status tc_init(spts_ctx* ctx) {
  spts_status s = tc_gemm_init(ctx);
  if (s != SPTS_OK) return s;
  if (cudaFuncSetAttribute(tc_attention_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, AP_SMEM) != cudaSuccess)
    return SPTS_ERR_CUDA;
  return SPTS_OK;
}

// The same kernel over a packed batch: Q [n_act, H*128], K [n_act, Hkv*128] and O hold the sequences' active rows one
// after the other, Vt [Hkv*128, ldvt] their transposed values with every sequence starting on a multiple of 8
// columns; `tiles` (device, n_tiles entries) lists every sequence's query tiles (tile pairs for odd GQA groups).
spts_status launch_tc_attention_packed(spts_ctx* ctx, const bf16* Q, const bf16* K, const bf16* Vt, int ldvt, int n_act,
                                       int vt_cols, const int4* tiles, int n_tiles, bf16* O) {
  if (n_tiles <= 0) return SPTS_OK;
  const auto& d = ctx->desc;
  if (d.head_dim != TILE || ctx->encode_tiled == nullptr) return SPTS_ERR_UNSUPPORTED;
  if (ldvt % 8) return SPTS_ERR_SHAPE;
  const int HD = d.n_q_heads * TILE, KD = d.n_kv_heads * TILE;
  CUtensorMap tmQ, tmK, tmV;
  if (!make_map(ctx, &tmQ, Q, (uint64_t)n_act, (uint64_t)HD, (uint64_t)HD)) return SPTS_ERR_CUDA;
  if (!make_map(ctx, &tmK, K, (uint64_t)n_act, (uint64_t)KD, (uint64_t)KD)) return SPTS_ERR_CUDA;
  if (!make_map(ctx, &tmV, Vt, (uint64_t)KD, (uint64_t)vt_cols, (uint64_t)ldvt)) return SPTS_ERR_CUDA;
  AttnParams p;
  p.m = 0; p.H = d.n_q_heads; p.Hkv = d.n_kv_heads; p.O = O; p.status = ctx->ws.status; p.tiles = tiles;
  p.pair_tiles = (d.n_q_heads / d.n_kv_heads) % 2 == 0 ? 0 : 1;
  dim3 grid(p.pair_tiles ? d.n_q_heads : d.n_q_heads / 2, n_tiles);
  tc_attention_pair_kernel<<<grid, AP_THREADS, AP_SMEM, ctx->stream>>>(tmQ, tmK, tmV, p);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status launch_tc_attention(spts_ctx* ctx, const bf16* Q, const bf16* K, const bf16* V, const bf16* Vt, int ldvt,
                                int m, bf16* O) {
  (void)V;
  if (m <= 0) return SPTS_OK;
  const auto& d = ctx->desc;
  if (d.head_dim != TILE || ctx->encode_tiled == nullptr) return SPTS_ERR_UNSUPPORTED;
  if (ldvt % 8) return SPTS_ERR_SHAPE;
  const int HD = d.n_q_heads * TILE, KD = d.n_kv_heads * TILE;
  CUtensorMap tmQ, tmK, tmV;
  if (!make_map(ctx, &tmQ, Q, (uint64_t)m, (uint64_t)HD, (uint64_t)HD)) return SPTS_ERR_CUDA;
  if (!make_map(ctx, &tmK, K, (uint64_t)m, (uint64_t)KD, (uint64_t)KD)) return SPTS_ERR_CUDA;
  if (!make_map(ctx, &tmV, Vt, (uint64_t)KD, (uint64_t)m, (uint64_t)ldvt)) return SPTS_ERR_CUDA;
  AttnParams p;
  p.m = m; p.H = d.n_q_heads; p.Hkv = d.n_kv_heads; p.pair_tiles = 0; p.O = O; p.status = ctx->ws.status; p.tiles = nullptr;
  // two score tiles per CTA: two heads of one KV head when the GQA group is even, else two query tiles of a head
  p.pair_tiles = (d.n_q_heads / d.n_kv_heads) % 2 == 0 ? 0 : 1;
  dim3 grid(p.pair_tiles ? d.n_q_heads : d.n_q_heads / 2,
            p.pair_tiles ? ceil_div(ceil_div(m, TILE), 2) : ceil_div(m, TILE));
  tc_attention_pair_kernel<<<grid, AP_THREADS, AP_SMEM, ctx->stream>>>(tmQ, tmK, tmV, p);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

}  // namespace spts
