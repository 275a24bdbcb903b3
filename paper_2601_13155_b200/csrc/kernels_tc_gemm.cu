// bf16 GEMM on the 5th-generation tensor cores with the SPTS epilogues fused in:
//
//   acc[i, j] = sum_k A[src(i), k] * W[j, k]          A rows optionally gathered by an index list
//
// Persistent, warp-specialised CTA (one per SM):
//   warp 0      TMA producer: W tile(s) and, when A is contiguous, the A tile
//   warps 6-9   (gather variant only) fetch the rows X[T_active, :] of the reduced attention / FFN
//               blocks (Algorithm 1, X^ = X[T_active, :]) straight into the 128B-swizzled operand
//               layout, so the gather costs no pass of its own
//   warp 1      TMEM allocation and the single-thread tcgen05.mma issue loop
//   warps 2-5   epilogue: tcgen05.ld of the fp32 accumulator (each warp its lane quarter, one
//               row per thread), then one of
//                 TC_STORE   out = bf16(acc * rstd[row])            (+ transposed copy for V)
//                 TC_ROPE    rotary embedding on 128-wide heads; optional PAP logits q_h . k
//                            from the unrounded keys (Eq. 4)
//                 TC_SWIGLU  tile = 128 gate | 128 up columns; out = bf16(silu(g) * u)   (Eq. 6)
//                 TC_RESID   X[dst(i), :] += acc, in place (Eq. 2 residual scatter)
//                 TC_SUMSQ   per-row sum of squares of the tile (Eq. 13), no matrix written
//                 TC_QFORM   per-row dot product of the tile with the row's own A operand (Eq. 13 as t G t^T)
// Accumulators are double-buffered in TMEM so the epilogue of tile t overlaps the MMAs of t+1.
#include "spts_common.cuh"
#include "tc_ptx.cuh"

namespace spts {

namespace {

using namespace ptx;

constexpr int BM = 128;
constexpr int BK = 64;                        // 64 bf16 = one 128-byte swizzle row
constexpr int A_STAGE_BYTES = BM * BK * 2;    // 16 KiB
constexpr int GEMM_THREADS = 192;
constexpr double RASTER_L2_BYTES = 48e6;       // how much of the grouped operand is allowed to sit in L2

template <int BN> struct Cfg {
  static constexpr int B_STAGE_BYTES = BN * BK * 2;
  static constexpr int STAGES = (BN == 256) ? 4 : 6;
  static constexpr int SMEM_BYTES = STAGES * (A_STAGE_BYTES + B_STAGE_BYTES) + 1024 + 256;
  static constexpr int TMEM_COLS = 2 * BN;
};
// The rotary epilogue stages, per epilogue warp, the (cos, sin) pairs of its 32 rows for half the frequencies:
// 32 rows x 256 bytes x 4 warps, after the barrier block.
constexpr int ROPE_STAGE_BYTES = 4 * 32 * 256;
template <int BN, int EPI> constexpr int gemm_smem_bytes() {
  return Cfg<BN>::SMEM_BYTES + (EPI == TC_ROPE ? ROPE_STAGE_BYTES : 0);
}

struct TcParams {
  const int32_t* idx;
  const int32_t* dst_idx;
  int M, Nout, K, a_rows;
  const void* a_ptr; int lda;   // A base and row stride (elements) for the gather producers
  const float* rowscale;
  bf16* out; int ldo;
  bf16* out_t; int ldt;
  const float2* cs;             // rotary table [rows, 64]
  const float* q; float* logits; int ld_logits; int group;
  const int32_t* row_seq; int q_stride;   // packed batch: row -> sequence, and the distance between two sequences' q
  const int32_t* out_t_col;     // TC_STORE: column of out_t a row goes to (nullptr: the row's own number)
  float* csq; int csq_parts;
  float* out_f32;               // TC_STORE: write fp32 [M, ldo] instead of the bf16 tile
  float* sal_t; int ld_sal;     // TC_SWIGLU: write |silu(g) u| as fp32 [column, row] instead of the bf16 tile
  int* status;
  int num_m, num_n;
  int raster_group;             // tiles of the grouped dimension whose operand stays in L2 (8 or 16)
  int raster_n;                 // 0: groups of row tiles sweep all column tiles; 1: groups of column tiles sweep all rows
};

// Tile order.  The CTAs in flight at one time work on `group` tiles of one dimension times as many
// tiles of the other as fit, so the grouped operand stays in L2 while the other streams past it; which
// dimension is grouped is chosen by the launcher from the two operands' sizes.
__device__ __forceinline__ void tile_coords(int t, int num_m, int num_n, int raster_n, int group, int& mb, int& nb) {
  const int na = raster_n ? num_n : num_m;      // grouped dimension
  const int nbo = raster_n ? num_m : num_n;     // swept dimension
  const int per_group = group * nbo;
  const int g = t / per_group;
  const int rem = t - g * per_group;
  const int gs = min(group, na - g * group);
  const int a = g * group + rem % gs;
  const int b = rem / gs;
  mb = raster_n ? b : a;
  nb = raster_n ? a : b;
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ void unpack_bf16(uint32_t w, float& a, float& b) {
  a = __uint_as_float(w << 16);
  b = __uint_as_float(w & 0xFFFF0000u);
}

// 32 fp32 values -> 32 bf16 stored to p (64 bytes, 16-byte aligned), columns [c0, c0+32) clipped to ncols
__device__ __forceinline__ void store32_bf16(bf16* p, const float* v, int c0, int ncols) {
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    if (c0 + g * 8 < ncols) {
      uint4 w;
      w.x = pack_bf16(v[g * 8 + 0], v[g * 8 + 1]);
      w.y = pack_bf16(v[g * 8 + 2], v[g * 8 + 3]);
      w.z = pack_bf16(v[g * 8 + 4], v[g * 8 + 5]);
      w.w = pack_bf16(v[g * 8 + 6], v[g * 8 + 7]);
      *reinterpret_cast<uint4*>(p + g * 8) = w;
    }
  }
}

// 16-byte asynchronous copy global -> shared; src_bytes == 0 writes zeros
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

constexpr int GATHER_WARPS = 4;      // extra producer warps of the row-gather variant
constexpr int GATHER_LAG = 2;        // k-blocks a gather thread keeps in flight before publishing

// GATHER: the A rows are X[idx[i], :].  Warps 6..9 fetch them with 16-byte cp.async copies --
// eight lanes per 128-byte row slice, written straight into the swizzled operand layout -- while
// warp 0 keeps feeding W through TMA.
template <int BN, int EPI, bool GATHER>
__global__ void __launch_bounds__(GATHER ? GEMM_THREADS + 32 * GATHER_WARPS : GEMM_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmB2, const TcParams p) {
  using C = Cfg<BN>;
  constexpr int STAGES = C::STAGES;
  constexpr int NT = (EPI == TC_SWIGLU) ? BN / 2 : BN;   // output columns per tile
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sA = base;
  const uint32_t sB = base + STAGES * A_STAGE_BYTES;
  const uint32_t bars = sB + STAGES * C::B_STAGE_BYTES;          // 8-byte aligned barrier block
  const uint32_t full_bar = bars, empty_bar = bars + 8 * STAGES;
  const uint32_t tfull_bar = bars + 16 * STAGES, tempty_bar = tfull_bar + 16;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + STAGES * (A_STAGE_BYTES + C::B_STAGE_BYTES) + 16 * STAGES + 32);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint64_t t0 = globaltimer_ns();
  const int total_tiles = p.num_m * p.num_n;
  const int kblocks = (p.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar + 8 * s, GATHER ? 1 + 32 * GATHER_WARPS : 1);
      mbar_init(empty_bar + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar + 8 * b, 1); mbar_init(tempty_bar + 8 * b, 4); }
    fence_mbar_init();
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB);
    if (EPI == TC_SWIGLU) prefetch_tensormap(&tmB2);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32((const void*)tmem_slot), C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        int mb, nb;
        tile_coords(t, p.num_m, p.num_n, p.raster_n, p.raster_group, mb, nb);
        const int m0 = mb * BM, n0 = nb * NT;
        for (int kb = 0; kb < kblocks; ++kb) {
          ok = mbar_wait(empty_bar + 8 * stage, phase ^ 1, abort_flag, t0);
          if (!ok) break;
          mbar_expect_tx(full_bar + 8 * stage, (GATHER ? 0 : A_STAGE_BYTES) + C::B_STAGE_BYTES);
          const int k0 = kb * BK;
          const uint32_t a_dst = sA + stage * A_STAGE_BYTES, b_dst = sB + stage * C::B_STAGE_BYTES;
          if (!GATHER) tma_load_2d(a_dst, &tmA, full_bar + 8 * stage, k0, m0);
          tma_load_2d(b_dst, &tmB, full_bar + 8 * stage, k0, n0);
          if (EPI == TC_SWIGLU) tma_load_2d(b_dst + (BN / 2) * BK * 2, &tmB2, full_bar + 8 * stage, k0, n0);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (GATHER && warp >= 6) {
    // ------------------------------------------------------------------ row-gather producers
    // lane -> (row offset lane / 8 inside a group of four rows, 16-byte chunk lane % 8)
    const int pw = warp - 6;
    const int chunk = lane & 7;
    const bf16* Abase = reinterpret_cast<const bf16*>(p.a_ptr);
    int stage = 0; uint32_t phase = 0;      // stage being filled
    int pstage = 0;                         // next stage to publish
    int inflight = 0;                       // committed, unpublished k-blocks
    bool ok = true;
    for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
      int mb, nb;
      tile_coords(t, p.num_m, p.num_n, p.raster_n, p.raster_group, mb, nb);
      const int m0 = mb * BM;
      const bf16* rowp[8];
      uint32_t soff[8];
      bool rvalid[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int rt = pw * 32 + e * 4 + (lane >> 3);          // row inside the tile
        const int gi = m0 + rt;
        rvalid[e] = gi < p.M;
        const int src = rvalid[e] ? p.idx[gi] : 0;
        rowp[e] = Abase + (size_t)src * p.lda + chunk * 8;
        soff[e] = (uint32_t)(rt * 128 + ((chunk ^ (rt & 7)) << 4));
      }
      for (int kb = 0; kb < kblocks; ++kb) {
        ok = mbar_wait(empty_bar + 8 * stage, phase ^ 1, abort_flag, t0);
        if (!ok) break;
        const int k0 = kb * BK;
        const bool kin = k0 + chunk * 8 < p.K;
        const uint32_t a_dst = sA + stage * A_STAGE_BYTES;
#pragma unroll
        for (int e = 0; e < 8; ++e) cp_async16(a_dst + soff[e], rowp[e] + k0, (rvalid[e] && kin) ? 16u : 0u);
        cp_async_commit();
        ++inflight;
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
        if (inflight > GATHER_LAG) {
          cp_async_wait<GATHER_LAG>();
          fence_proxy_async_smem();
          mbar_arrive(full_bar + 8 * pstage);
          if (++pstage == STAGES) pstage = 0;
          --inflight;
        }
      }
    }
    cp_async_wait<0>();
    fence_proxy_async_smem();
    while (ok && inflight > 0) {
      mbar_arrive(full_bar + 8 * pstage);
      if (++pstage == STAGES) pstage = 0;
      --inflight;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16(BM, BN);
      int stage = 0; uint32_t phase = 0;
      int abuf = 0; uint32_t aphase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        ok = mbar_wait(tempty_bar + 8 * abuf, aphase ^ 1, abort_flag, t0);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + abuf * BN;
        for (int kb = 0; kb < kblocks; ++kb) {
          ok = mbar_wait(full_bar + 8 * stage, phase, abort_flag, t0);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_addr = sA + stage * A_STAGE_BYTES, b_addr = sB + stage * C::B_STAGE_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            mma_bf16(d_tmem, smem_desc_sw128(a_addr + k * 32), smem_desc_sw128(b_addr + k * 32), idesc,
                     (kb > 0 || k > 0) ? 1u : 0u);
          }
          mma_commit(empty_bar + 8 * stage);          // frees the smem stage when these MMAs finish
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        mma_commit(tfull_bar + 8 * abuf);             // accumulator complete
        if (++abuf == 2) { abuf = 0; aphase ^= 1; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int quarter = warp & 3;
    const int row_in_tile = quarter * 32 + lane;
    int abuf = 0; uint32_t aphase = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
      int mb, nb;
      tile_coords(t, p.num_m, p.num_n, p.raster_n, p.raster_group, mb, nb);
      const int grow = mb * BM + row_in_tile;
      const int n0 = nb * NT;
      const bool row_ok = grow < p.M;
      int src = 0;
      float rs = 1.0f;
      if (row_ok) {
        src = p.idx ? p.idx[grow] : grow;
        if (p.rowscale) rs = p.rowscale[src];
      }
      ok = mbar_wait(tfull_bar + 8 * abuf, aphase, abort_flag, t0);
      if (!ok) break;
      tc_fence_after();
      const uint32_t tacc = tmem_base + abuf * BN + ((uint32_t)(quarter * 32) << 16);

      if (EPI == TC_STORE) {
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          tmem_ld32(tacc + c, r);
          tmem_ld_wait();
          if (row_ok && n0 + c < p.Nout) {
            float v[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]) * rs;
            if (p.out_f32 != nullptr) {            // unrounded fp32 result (probe logits of the query window)
              float* o = p.out_f32 + (size_t)grow * p.ldo + n0 + c;
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (n0 + c + i < p.Nout) o[i] = v[i];
              continue;
            }
            store32_bf16(p.out + (size_t)grow * p.ldo + n0 + c, v, n0 + c, p.Nout);
            if (p.out_t != nullptr) {
              const int tcol = p.out_t_col ? p.out_t_col[grow] : grow;
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (n0 + c + i < p.Nout) p.out_t[(size_t)(n0 + c + i) * p.ldt + tcol] = __float2bfloat16_rn(v[i]);
            }
          }
        }
      } else if (EPI == TC_ROPE) {
        // Rotary embedding on the 128-wide heads of the tile (and, for the probe, the logits q_h . k of Eq. 4 from
        // the unrounded keys).  The table row of a token (64 (cos, sin) pairs, 512 bytes) is the same for every head
        // and every column tile; read per lane it is a 32-line gather per load, and that gather cost 11 % of the
        // gathered Q projection.  So each warp stages its 32 rows' pairs for one half of the frequencies in shared
        // memory -- two rows per load instruction, 16 lanes x 16 bytes each, fully used sectors -- and both heads of
        // the tile read them from there (16-byte chunks XOR-swizzled by the row so that neither the staging stores
        // nor the per-row reads conflict).
        const float inv_sqrt_d = 0.08838834764831845f;   // 1 / sqrt(128)
        constexpr int NH = BN / 128;                     // heads per tile
        uint8_t* stage = gen + STAGES * (A_STAGE_BYTES + C::B_STAGE_BYTES) + 256 + quarter * (32 * 256);
        float dots[NH][8];
#pragma unroll
        for (int hh = 0; hh < NH; ++hh)
#pragma unroll
          for (int g = 0; g < 8; ++g) dots[hh][g] = 0.f;
#pragma unroll 1
        for (int jj = 0; jj < 2; ++jj) {
          __syncwarp();                                  // the previous half's readers are done
          {
            float4 v[16];                                // all 16 loads in flight before the first store
#pragma unroll
            for (int k = 0; k < 16; ++k) {
              const int r = 2 * k + (lane >> 4);
              const int srow = __shfl_sync(0xffffffffu, src, r);
              const int rok = __shfl_sync(0xffffffffu, (int)row_ok, r);
              v[k] = make_float4(1.f, 0.f, 1.f, 0.f);
              if (rok) v[k] = __ldg(reinterpret_cast<const float4*>(p.cs) + (size_t)srow * 32 + jj * 16 + (lane & 15));
            }
#pragma unroll
            for (int k = 0; k < 16; ++k) {
              const int r = 2 * k + (lane >> 4), ch = lane & 15;
              *reinterpret_cast<float4*>(stage + r * 256 + ((ch ^ (r & 15)) << 4)) = v[k];
            }
          }
          __syncwarp();
#pragma unroll
          for (int hh = 0; hh < NH; ++hh) {
            const int hcol = n0 + hh * 128;               // first column of this head
            uint32_t lo[32], hi[32];
            tmem_ld32(tacc + hh * 128 + jj * 32, lo);
            tmem_ld32(tacc + hh * 128 + 64 + jj * 32, hi);
            tmem_ld_wait();
            if (row_ok && hcol < p.Nout) {
              float a[32], b[32];
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                // (cos, sin) of two consecutive frequencies
                const float4 c2 = *reinterpret_cast<const float4*>(stage + lane * 256 + ((((i >> 1)) ^ (lane & 15)) << 4));
                float x0 = __uint_as_float(lo[i]) * rs, y0 = __uint_as_float(hi[i]) * rs;
                float x1 = __uint_as_float(lo[i + 1]) * rs, y1 = __uint_as_float(hi[i + 1]) * rs;
                a[i] = x0 * c2.x - y0 * c2.y;
                b[i] = y0 * c2.x + x0 * c2.y;
                a[i + 1] = x1 * c2.z - y1 * c2.w;
                b[i + 1] = y1 * c2.z + x1 * c2.w;
              }
              bf16* o = p.out + (size_t)grow * p.ldo + hcol + jj * 32;
              store32_bf16(o, a, 0, 32);
              store32_bf16(o + 64, b, 0, 32);
              if (p.logits != nullptr) {
                const int kvh = hcol >> 7;
                // packed batch: every sequence is probed with its own last token's query
                const float* qseq = p.q + (p.row_seq ? (size_t)p.row_seq[src] * p.q_stride : 0);
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                  if (g < p.group) {
                    const float* qh = qseq + (size_t)(kvh * p.group + g) * 128 + jj * 32;
                    float d = dots[hh][g];
#pragma unroll
                    for (int i = 0; i < 32; ++i) d = fmaf(a[i], __ldg(qh + i), fmaf(b[i], __ldg(qh + 64 + i), d));
                    dots[hh][g] = d;
                  }
                }
                // query heads beyond the eight kept in registers (GQA groups larger than 8): their partial sums
                // over this half of the frequencies go through the logits row itself (same thread, same address)
                for (int g = 8; g < p.group; ++g) {
                  const float* qh = qseq + (size_t)(kvh * p.group + g) * 128 + jj * 32;
                  float d = 0.f;
#pragma unroll
                  for (int i = 0; i < 32; ++i) d = fmaf(a[i], __ldg(qh + i), fmaf(b[i], __ldg(qh + 64 + i), d));
                  float* lp = p.logits + (size_t)(kvh * p.group + g) * p.ld_logits + grow;
                  *lp = jj == 0 ? d : (*lp + d) * inv_sqrt_d;
                }
              }
            }
          }
        }
        if (p.logits != nullptr && row_ok) {
#pragma unroll
          for (int hh = 0; hh < NH; ++hh) {
            const int hcol = n0 + hh * 128;
            if (hcol < p.Nout) {
              const int kvh = hcol >> 7;
#pragma unroll
              for (int g = 0; g < 8; ++g)
                if (g < p.group) p.logits[(size_t)(kvh * p.group + g) * p.ld_logits + grow] = dots[hh][g] * inv_sqrt_d;
            }
          }
        }
      } else if (EPI == TC_SWIGLU) {
#pragma unroll 1
        for (int c = 0; c < BN / 2; c += 32) {
          uint32_t g[32], u[32];
          tmem_ld32(tacc + c, g);
          tmem_ld32(tacc + BN / 2 + c, u);
          tmem_ld_wait();
          if (row_ok && n0 + c < p.Nout) {
            float v[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              float a = __uint_as_float(g[i]) * rs, b = __uint_as_float(u[i]) * rs;
              v[i] = __fdividef(a, 1.0f + __expf(-a)) * b;   // fast exp / divide: ~1e-6 relative, far below the bf16 store
            }
            if (p.sal_t != nullptr) {
              // saliency of the proxy construction: |silu(g) * u| in fp32, one row per channel (transposed)
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (n0 + c + i < p.Nout) p.sal_t[(size_t)(n0 + c + i) * p.ld_sal + grow] = fabsf(v[i]);
            } else {
              store32_bf16(p.out + (size_t)grow * p.ldo + n0 + c, v, n0 + c, p.Nout);
            }
          }
        }
      } else if (EPI == TC_RESID) {
        int dst = grow;
        if (row_ok && p.dst_idx) dst = p.dst_idx[grow];
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          tmem_ld32(tacc + c, r);
          tmem_ld_wait();
          if (row_ok && n0 + c < p.Nout) {
            bf16* xp = p.out + (size_t)dst * p.ldo + n0 + c;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              if (n0 + c + g * 8 < p.Nout) {
                uint4 w = *reinterpret_cast<const uint4*>(xp + g * 8);
                uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  float x0, x1;
                  unpack_bf16(ww[e], x0, x1);
                  ww[e] = pack_bf16(x0 + __uint_as_float(r[g * 8 + 2 * e]), x1 + __uint_as_float(r[g * 8 + 2 * e + 1]));
                }
                *reinterpret_cast<uint4*>(xp + g * 8) = make_uint4(ww[0], ww[1], ww[2], ww[3]);
              }
            }
          }
        }
      } else if (EPI == TC_QFORM) {
        // Eq. 13 through the Gram matrix: the tile holds y = t [G_hi ; G_lo]^T for this row's t (the A operand itself,
        // r wide); its share of t G t^T is sum_j y_j t_{j mod r}.  No matrix is written.
        float s = 0.f;
        const bf16* trow = reinterpret_cast<const bf16*>(p.a_ptr) + (size_t)grow * p.lda;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          tmem_ld32(tacc + c, r);
          tmem_ld_wait();
          if (row_ok && n0 + c < p.Nout) {
            const int k0 = (n0 + c) % p.K;               // K = r, a multiple of 32: the 32 columns stay inside one copy
            const uint4* tp = reinterpret_cast<const uint4*>(trow + k0);
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              const uint4 w = __ldg(tp + g);
              const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                float t0v, t1v;
                unpack_bf16(ww[e], t0v, t1v);
                s = fmaf(__uint_as_float(r[g * 8 + 2 * e]), t0v, s);
                s = fmaf(__uint_as_float(r[g * 8 + 2 * e + 1]), t1v, s);
              }
            }
          }
        }
        if (row_ok) p.csq[(size_t)grow * p.csq_parts + nb] = s;
      } else {   // TC_SUMSQ
        float s = 0.f;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          tmem_ld32(tacc + c, r);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            float v = __uint_as_float(r[i]);
            if (n0 + c + i < p.Nout) s = fmaf(v, v, s);
          }
        }
        if (row_ok) p.csq[(size_t)grow * p.csq_parts + nb] = s;
      }
      // accumulator buffer drained: hand it back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar + 8 * abuf);
      if (++abuf == 2) { abuf = 0; aphase ^= 1; }
    }
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // a wait ran out: give copies still in flight time to land before shared memory is released
    if (threadIdx.x == 0) set_status(p.status, SPTS_ERR_TIMEOUT);
    const uint64_t t1 = globaltimer_ns();
    while (globaltimer_ns() - t1 < 200000ull) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

// The give-up path of the bounded waits on its own: two roles wait on barriers nobody arrives on.  Warp 0's wait
// runs into the (shortened) limit and raises the abort flag; warp 1's wait has a limit far away and must return
// because of the flag.  Then the same teardown as the kernels above: status word, drain delay, normal exit.
__global__ void __launch_bounds__(64, 1) wait_selftest_kernel(uint64_t limit_ns, int* status, int* observed) {
  __shared__ __align__(8) uint64_t bar_store[2];
  __shared__ int abort_store;
  volatile int* abort_flag = &abort_store;
  const uint32_t bar0 = smem_u32(&bar_store[0]), bar1 = smem_u32(&bar_store[1]);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint64_t t0 = globaltimer_ns();
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(bar0, 1);
    mbar_init(bar1, 1);
    fence_mbar_init();
  }
  __syncthreads();
  if (lane == 0) {
    const bool ok = warp == 0 ? mbar_wait(bar0, 0, abort_flag, t0, limit_ns) : mbar_wait(bar1, 0, abort_flag, t0);
    observed[warp] = ok ? 1 : 2;            // 2 = the wait was abandoned
  }
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) set_status(status, SPTS_ERR_TIMEOUT);
    const uint64_t t1 = globaltimer_ns();
    while (globaltimer_ns() - t1 < 200000ull) { }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D bf16 tensor [rows, cols] with row stride ld (elements), box [box_rows, 64 cols], 128B swizzle.
bool make_map(spts_ctx* ctx, CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint64_t ld,
              uint32_t box_rows) {
  EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstride[1] = {ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int BN, int EPI, bool GATHER>
spts_status launch_one_g(spts_ctx* ctx, const TcGemmArgs& a) {
  constexpr int NT = (EPI == TC_SWIGLU) ? BN / 2 : BN;
  TcParams p;
  p.idx = a.idx; p.dst_idx = a.dst_idx; p.M = a.M; p.Nout = a.Nout; p.K = a.K; p.a_rows = a.a_rows;
  p.a_ptr = a.A; p.lda = a.lda;
  p.rowscale = a.rowscale; p.out = a.out; p.ldo = a.ldo; p.out_t = a.out_t; p.ldt = a.ldt;
  p.cs = ctx->ws.rope_cs; p.q = a.q; p.logits = a.logits; p.ld_logits = a.ld_logits; p.group = a.group;
  p.csq = a.csq; p.csq_parts = a.csq_parts; p.status = ctx->ws.status;
  p.sal_t = a.sal_t; p.ld_sal = a.ld_sal; p.out_f32 = a.out_f32;
  p.row_seq = a.row_seq; p.q_stride = a.q_stride; p.out_t_col = a.out_t_col;
  p.num_m = ceil_div(a.M, BM);
  p.num_n = ceil_div(a.Nout, NT);
  {
    // DRAM traffic of the candidate tile orders: the grouped operand is read once per group (it must fit in
    // L2 beside the streams), the other operand once per pass over the groups
    const double a_bytes = 2.0 * a.M * a.K, w_bytes = 2.0 * a.Nout * a.K * (EPI == TC_SWIGLU ? 2.0 : 1.0);
    double best = -1.0;
    for (int rn = 0; rn < 2; ++rn) {
      for (int grp = 8; grp <= 16; grp += 8) {
        const int tiles = rn ? p.num_n : p.num_m;
        const double band = (rn ? w_bytes / p.num_n : a_bytes / p.num_m) * grp;
        if (grp > 8 && band > RASTER_L2_BYTES) continue;
        const double cost = (double)ceil_div(tiles, grp) * (rn ? a_bytes : w_bytes) + (rn ? w_bytes : a_bytes);
        if (best < 0.0 || cost < best) { best = cost; p.raster_n = rn; p.raster_group = grp; }
      }
    }
  }
  CUtensorMap tmA, tmB, tmB2;
  if (!make_map(ctx, &tmA, a.A, (uint64_t)a.a_rows, (uint64_t)a.K, (uint64_t)a.lda, (uint32_t)BM)) return SPTS_ERR_CUDA;
  if (!make_map(ctx, &tmB, a.W, (uint64_t)a.Nout, (uint64_t)a.K, (uint64_t)(a.ldw ? a.ldw : a.K), (uint32_t)NT)) return SPTS_ERR_CUDA;
  if (EPI == TC_SWIGLU) {
    if (!make_map(ctx, &tmB2, a.W2, (uint64_t)a.Nout, (uint64_t)a.K, (uint64_t)a.K, (uint32_t)NT)) return SPTS_ERR_CUDA;
  } else {
    tmB2 = tmB;
  }
  const int tiles = p.num_m * p.num_n;
  const int grid = tiles < ctx->sm_count ? tiles : ctx->sm_count;
  tc_gemm_kernel<BN, EPI, GATHER><<<grid, GATHER ? GEMM_THREADS + 32 * GATHER_WARPS : GEMM_THREADS, gemm_smem_bytes<BN, EPI>(),
                                    ctx->stream>>>(tmA, tmB, tmB2, p);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

template <int BN, int EPI>
spts_status launch_one(spts_ctx* ctx, const TcGemmArgs& a) {
  if (EPI == TC_STORE || EPI == TC_ROPE || EPI == TC_SWIGLU) {
    if (a.idx != nullptr) return launch_one_g<BN, EPI, (EPI == TC_STORE || EPI == TC_ROPE || EPI == TC_SWIGLU)>(ctx, a);
  } else if (a.idx != nullptr) {
    return SPTS_ERR_UNSUPPORTED;
  }
  return launch_one_g<BN, EPI, false>(ctx, a);
}

template <int BN, int EPI>
bool set_smem_attr() {
  bool ok = cudaFuncSetAttribute(tc_gemm_kernel<BN, EPI, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 gemm_smem_bytes<BN, EPI>()) == cudaSuccess;
  if (EPI == TC_STORE || EPI == TC_ROPE || EPI == TC_SWIGLU)
    ok = ok && cudaFuncSetAttribute(tc_gemm_kernel<BN, EPI, (EPI == TC_STORE || EPI == TC_ROPE || EPI == TC_SWIGLU)>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize, gemm_smem_bytes<BN, EPI>()) == cudaSuccess;
  return ok;
}

}  // namespace

int tc_sumsq_parts(int n_out) { return ceil_div(n_out, 256); }

spts_status launch_wait_selftest(spts_ctx* ctx, uint32_t limit_us) {
  // observed[] lives behind the status word: ws.status has 64 ints, the first is the status itself
  wait_selftest_kernel<<<1, 64, 0, ctx->stream>>>((uint64_t)limit_us * 1000ull, ctx->ws.status, ctx->ws.status + 8);
  SPTS_CUDA_OK(ctx);
  return SPTS_OK;
}

spts_status tc_gemm_init(spts_ctx* ctx) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || fn == nullptr)
    return SPTS_ERR_CUDA;
  ctx->encode_tiled = fn;
  bool ok = set_smem_attr<256, TC_STORE>() && set_smem_attr<256, TC_ROPE>() && set_smem_attr<256, TC_SWIGLU>() &&
            set_smem_attr<256, TC_RESID>() && set_smem_attr<256, TC_SUMSQ>() && set_smem_attr<128, TC_STORE>() &&
            set_smem_attr<128, TC_ROPE>() && set_smem_attr<128, TC_SWIGLU>() && set_smem_attr<256, TC_QFORM>();
  return ok ? SPTS_OK : SPTS_ERR_CUDA;
}

spts_status launch_tc_gemm(spts_ctx* ctx, int epi, const TcGemmArgs& a) {
  if (a.M <= 0) return SPTS_OK;
  if (ctx->encode_tiled == nullptr) return SPTS_ERR_UNSUPPORTED;
  if ((a.K % 8) || (a.lda % 8) || (reinterpret_cast<uintptr_t>(a.A) & 15) || (reinterpret_cast<uintptr_t>(a.W) & 15))
    return SPTS_ERR_SHAPE;
  if (a.out == nullptr && epi != TC_SUMSQ && epi != TC_QFORM && !(epi == TC_SWIGLU && a.sal_t != nullptr) &&
      !(epi == TC_STORE && a.out_f32 != nullptr))
    return SPTS_ERR_INVALID_ARG;
  if (a.ldw % 8) return SPTS_ERR_SHAPE;
  if (a.out != nullptr && ((a.ldo % 8) || (reinterpret_cast<uintptr_t>(a.out) & 15))) return SPTS_ERR_SHAPE;
  if ((a.Nout % 8) && a.out_f32 == nullptr) return SPTS_ERR_SHAPE;
  const bool narrow = a.Nout <= 128;       // a 128-wide tile wastes less on the skinny proxy factors
  // A skinny output (the proxy's stacked first factors: 2r columns) gives one 256-wide tile per 128 rows, and the
  // tile count then rounds badly against the SM count (256 tiles on 148 SMs: two waves, the second 73 % idle).
  // Half-width tiles double the count; take them when they fill the waves clearly better.
  bool half = false;
  if (epi == TC_STORE && !narrow && a.Nout <= 512) {
    const int sm = ctx->sm_count > 0 ? ctx->sm_count : 148;
    const int t256 = ceil_div(a.M, BM) * ceil_div(a.Nout, 256), t128 = ceil_div(a.M, BM) * ceil_div(a.Nout, 128);
    const double e256 = (double)t256 / ((double)ceil_div(t256, sm) * sm), e128 = (double)t128 / ((double)ceil_div(t128, sm) * sm);
    half = e128 > e256 + 0.08;
  }
  switch (epi) {
    case TC_STORE: return (narrow || half) ? launch_one<128, TC_STORE>(ctx, a) : launch_one<256, TC_STORE>(ctx, a);
    case TC_ROPE:
      if (a.Nout % 128) return SPTS_ERR_SHAPE;
      return narrow ? launch_one<128, TC_ROPE>(ctx, a) : launch_one<256, TC_ROPE>(ctx, a);
    case TC_SWIGLU: return (a.Nout <= 64) ? launch_one<128, TC_SWIGLU>(ctx, a) : launch_one<256, TC_SWIGLU>(ctx, a);
    case TC_RESID: return launch_one<256, TC_RESID>(ctx, a);
    case TC_SUMSQ: return launch_one<256, TC_SUMSQ>(ctx, a);
    case TC_QFORM:
      if (a.K % 32 || a.Nout % a.K || a.idx != nullptr) return SPTS_ERR_SHAPE;
      return launch_one<256, TC_QFORM>(ctx, a);
    default: return SPTS_ERR_INVALID_ARG;
  }
}

}  // namespace spts
