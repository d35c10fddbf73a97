// bf16 GEMM on the 5th-generation tensor cores (tcgen05), fp32 accumulation in TMEM.
//
//   out[b, m, n] = epilogue( sum_k A[b, m, k] * B[b, n, k] )
//
// Both operands are read "reduction dimension contiguous" (Section 3.2.2) straight from the
// producer's buffer: the composed index map of an eliminated layout run is affine here, so it
// becomes a TMA tensor map (up to 5-D box) and costs nothing at run time.  An operand whose
// rows -- not its reduction dimension -- are contiguous in the producer's buffer (the NCHW ->
// NHWC case) is loaded as it lies and multiplied through the MN-major operand mode of the
// tensor core, so that transpose disappears as well.
//
// Persistent CTAs (one per SM) of 19 warps: warp 0 issues TMA loads into a 3- to 6-stage shared-memory
// ring (a second producer warp takes the B operand when the reduction is long), warp 1 owns the TMEM
// allocation and issues tcgen05.mma (one thread) into one of two accumulator buffers, warps 2-17 run
// the epilogue of the previous tile meanwhile (TMEM -> registers -> bias / GELU / RoPE / residual ->
// bf16 -> staged whole-row stores, optionally scattering rows through an index map: window reverse +
// reverse cyclic shift folded into the store).
#include <mutex>
#include <unordered_map>
#include <string>
#include <vector>

#include "gemm_tc.cuh"
#include "ptx.cuh"


namespace smartmem {
namespace {

constexpr int BM = 128;
constexpr int BK = 64;                   // 64 bf16 = 128 bytes = one swizzle row
constexpr int A_STAGE_BYTES = BM * BK * 2;

struct OpCoord {
  int rank, mn_major;
  FastDiv tiles_inner;
  int n_outer;                           // outer row atoms then batch atoms, innermost first
  int n_outer_row;
  FastDiv outer[3];
};

struct GemmArgs {
  int M, N, K;
  int tiles_n, tiles_m, batch;
  FastDiv fd_tiles_n, fd_tiles_m;        // tile index -> (tile_n, tile_m, batch) without hardware division
  OpCoord ca, cb;
  __nv_bfloat16* out;
  long long ldc, out_batch_stride;
  const __nv_bfloat16* bias;
  const __nv_bfloat16* residual;
  int gelu, has_rowmap;
  int rope_cols, rope_S, rope_pos0;      // columns [0, rope_cols) are rotated; position = rope_pos0 + row % rope_S
  int rope_half;                         // R / 2: the first R columns of each 128-wide head rotate, pairs (i, i + R/2)
  float rope_c;                          // log2(theta) / (R / 2)
  int seg_cols;                          // > 0: column segment s of a row goes to seg_out[s] + row * seg_ld[s]
  __nv_bfloat16* seg_out[3];
  long long seg_ld[3];
  __nv_bfloat16* out2;                   // second copy of the result, transposed inside groups of out2_S rows (null: none)
  FastDiv fd_out2_S;
  int* status;
  int tma_out;                           // lean epilogue: the output leaves as TMA boxes (tensor map tmC) instead of per-thread stores
  DevMap rowmap;
};

// Tile -> TMA coordinates of an operand: row origin inside the innermost row atom and the digits
// of the outer row atoms / batch atoms (every tensor map is padded to rank 5, so all five
// coordinates always exist and stay in registers).
struct TileCoord {
  int row0, o0, o1, o2;
};
__device__ __forceinline__ TileCoord op_coords(const OpCoord& oc, uint32_t tile, uint32_t batch, int tile_rows) {
  uint32_t q = fd_div(tile, oc.tiles_inner);
  TileCoord tc;
  tc.row0 = (int)(tile - q * oc.tiles_inner.d) * tile_rows;
  int o[3] = {0, 0, 0};
#pragma unroll
  for (int i = 0; i < 3; ++i) {
    if (i < oc.n_outer) {
      const bool from_rows = i < oc.n_outer_row;
      const uint32_t src = from_rows ? q : batch;
      const uint32_t qq = fd_div(src, oc.outer[i]);
      o[i] = (int)(src - qq * oc.outer[i].d);
      if (from_rows) q = qq; else batch = qq;
    }
  }
  tc.o0 = o[0]; tc.o1 = o[1]; tc.o2 = o[2];
  return tc;
}
__device__ __forceinline__ void tma_load_op(const OpCoord& oc, void* dst, const CUtensorMap* tm, uint64_t* bar, int k0,
                                            int row0, const TileCoord& tc) {
  ptx::tma_load_5d(dst, tm, bar, oc.mn_major ? row0 : k0, oc.mn_major ? k0 : row0, tc.o0, tc.o1, tc.o2);
}
// CTA pair: the bytes are counted on the even CTA's barrier (a shared::cluster address)
__device__ __forceinline__ void tma_load_op_pair(const OpCoord& oc, void* dst, const CUtensorMap* tm, uint32_t bar_cluster, int k0,
                                                 int row0, const TileCoord& tc) {
  ptx::tma_load_5d_pair(dst, tm, bar_cluster, k0, row0, tc.o0, tc.o1, tc.o2);
}

struct TileIdx {
  uint32_t tile_n, tile_m, batch;
};
__device__ __forceinline__ TileIdx split_tile(uint32_t t, const FastDiv& fn, const FastDiv& fm) {
  const uint32_t r = fd_div(t, fn), b = fd_div(r, fm);
  return {t - r * fn.d, r - b * fm.d, b};
}

// GELU in the bf16 epilogue: u * Phi(u) with Phi evaluated through the hyperbolic-tangent form
// 0.5 (1 + tanh(sqrt(2/pi) (u + 0.044715 u^3))) and the hardware tanh.  It differs from the erf
// form by at most 5e-4 in absolute value, i.e. by less than an eighth of a bf16 ulp wherever the
// result exceeds 1 and by less than 1e-4 |u| near zero, at a third of the instruction count (the
// epilogue of the fc1 GEMM is issue-bound).  The fp32 kernels use erff.
__device__ __forceinline__ float gelu_fast(float u) {
  const float u2 = u * u;
  const float inner = u * fmaf(0.0356774081f, u2, 0.7978845608f);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(inner));
  const float h = 0.5f * u;
  return fmaf(h, t, h);
}

constexpr int kEpiWarps = 16;
constexpr int kThreads = 64 + 32 * kEpiWarps + 32;      // + a second TMA producer warp (B operand)

// Persistent kernel: one CTA per SM walks over output tiles (tile = blockIdx.x + i * gridDim.x).
// The shared-memory ring and two TMEM accumulator buffers run across tile boundaries, so the
// loads and MMAs of tile i+1 overlap the epilogue of tile i.
//
// PAIR: the two CTAs of a cluster share one 256 x BN tile (cta_group::2).  Each loads its own 128 rows of A and its own
// half of the B tile's rows -- two thirds of the operand bytes a lone CTA pulls in per product, which is what bounds a
// 128 x 256 tile (48 KB per k-block against the ~64 bytes per clock an SM takes in) -- and keeps its own 128 rows of the
// accumulator, which it drains itself.  The even CTA counts both CTAs' bytes on its `full` barriers, issues the products
// and signals `empty` / `tmem_full` in both CTAs; both CTAs' epilogue warps arrive on its `tmem_empty`.
// LEAN (pairs only): the epilogue knows bias and GELU only (no rotary embedding, residual or second copy), which leaves it
// the registers to pull its whole accumulator slice out of tensor memory at once and hand the buffer back before any
// arithmetic -- for short reductions, where a tile's products take no longer than its epilogue.
template <int BN, int STAGES, bool A_MN, bool PAIR, bool LEAN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmC, const __grid_constant__ GemmArgs g) {
  static_assert(!PAIR || ((BN == 256 || BN == 128) && !A_MN), "CTA pairs: 256- or 128-wide tiles, K-major A");
  static_assert(!LEAN || PAIR, "the lean epilogue comes with CTA pairs");
  constexpr int BN_CTA = PAIR ? BN / 2 : BN;               // rows of B this CTA loads
  constexpr int B_STAGE_BYTES = BN_CTA * BK * 2;
  constexpr uint32_t ACC_COLS = BN <= 32 ? 32 : BN <= 64 ? 64 : BN <= 128 ? 128 : 256;   // one accumulator buffer
  constexpr uint32_t TMEM_COLS = 2 * ACC_COLS;
  constexpr uint32_t IDESC = ptx::make_idesc_bf16(PAIR ? 2 * BM : BM, BN, A_MN, false);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  uint8_t* sA = smem;
  uint8_t* sB = smem + STAGES * A_STAGE_BYTES;
  // lean epilogue: a 32 x 32 output box per epilogue warp (64-byte rows, 64-byte swizzle), right behind the ring
  constexpr int CBOX_BYTES = 32 * 64;
  uint8_t* cstage = sB + STAGES * B_STAGE_BYTES;
  uint64_t* full = reinterpret_cast<uint64_t*>(cstage + (LEAN ? kEpiWarps * CBOX_BYTES : 0));
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;                      // [2]
  uint64_t* tmem_empty = tmem_full + 2;                      // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 2);
  int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);
  uint8_t* stage_base = reinterpret_cast<uint8_t*>(tmem_slot + 4);                      // 16-byte aligned

  const int warp = __shfl_sync(0xFFFFFFFFu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // (warp: provably uniform)
  const int nkb = (g.K + BK - 1) / BK;
  const int last_ksteps = (g.K - (nkb - 1) * BK + 15) / 16;
  const bool two_producers = nkb >= 8;
  const uint32_t total_tiles = (uint32_t)g.tiles_n * g.tiles_m * g.batch;   // PAIR: tiles_m counts 256-row tiles
  const uint32_t rank = PAIR ? ptx::cluster_ctarank() : 0u;                  // which half of the pair's tile
  const bool leader = rank == 0;
  const uint32_t cta_first = PAIR ? blockIdx.x >> 1 : blockIdx.x, cta_step = PAIR ? gridDim.x >> 1 : gridDim.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(&full[s], two_producers ? 2 : 1);  // one arrival per producer warp
      ptx::mbar_init(&empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(&tmem_full[b], 1);
      ptx::mbar_init(&tmem_empty[b], PAIR ? 2 * kEpiWarps : kEpiWarps);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
    if (LEAN && g.tma_out) ptx::prefetch_tensormap(&tmC);
  }
  if (warp == 1) {
    if constexpr (PAIR) ptx::tmem_alloc_pair(tmem_slot, TMEM_COLS);
    else ptx::tmem_alloc(tmem_slot, TMEM_COLS);
  }
  ptx::tc_fence_before();
  if constexpr (PAIR) {
    __syncwarp();
    ptx::cluster_sync();            // the peer's barriers are initialised before anything of this CTA signals them
  } else {
    __syncthreads();
  }
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                       // everything above overlapped the previous kernel's tail
  pdl_launch_dependents();

  if (warp == 0) {
    if (lane == 0) {
      uint32_t kbg = 0, s = 0, ph = 0;                       // k-block counter across tiles, ring position
      bool ok = true;
      uint32_t pit = 0;
      const uint32_t full0 = PAIR ? ptx::mapa(ptx::smem_u32(full), 0) : 0u;     // the even CTA's `full` barriers
      for (uint32_t t = cta_first; t < total_tiles && ok; t += cta_step, ++pit) {
        const TileIdx ti_ = split_tile(t, g.fd_tiles_n, g.fd_tiles_m);
        const uint32_t tile_n = ti_.tile_n, tile_m = PAIR ? 2 * ti_.tile_m + rank : ti_.tile_m, batch = ti_.batch;
        const TileCoord ta = op_coords(g.ca, tile_m, batch, BM), tb = op_coords(g.cb, tile_n, batch, BN);
        const int brow0 = tb.row0 + (int)rank * BN_CTA;
        for (int kb = 0; kb < nkb; ++kb, ++kbg) {
          ok = ptx::mbar_wait(&empty[s], ph ^ 1, abort_flag, g.status);
          if (!ok) break;
          if constexpr (PAIR) {
            if (leader) ptx::mbar_expect_tx(&full[s], 2 * (two_producers ? A_STAGE_BYTES : A_STAGE_BYTES + B_STAGE_BYTES));
            tma_load_op_pair(g.ca, sA + s * A_STAGE_BYTES, &tmA, full0 + s * 8, kb * BK, ta.row0, ta);
            if (!two_producers) tma_load_op_pair(g.cb, sB + s * B_STAGE_BYTES, &tmB, full0 + s * 8, kb * BK, brow0, tb);
          } else {
            ptx::mbar_expect_tx(&full[s], two_producers ? A_STAGE_BYTES : A_STAGE_BYTES + B_STAGE_BYTES);
            tma_load_op(g.ca, sA + s * A_STAGE_BYTES, &tmA, &full[s], kb * BK, ta.row0, ta);
            if (A_MN) tma_load_op(g.ca, sA + s * A_STAGE_BYTES + A_STAGE_BYTES / 2, &tmA, &full[s], kb * BK, ta.row0 + 64, ta);
            if (!two_producers) tma_load_op(g.cb, sB + s * B_STAGE_BYTES, &tmB, &full[s], kb * BK, tb.row0, tb);
          }
          if (++s == STAGES) { s = 0; ph ^= 1; }
        }
      }
      if (*abort_flag && PAIR) {
        // unwinding a pair: the copies of the odd CTA are counted on the even CTA's barriers, so each side just gives
        // whatever is in flight a fixed time to land
        const unsigned long long t0 = ptx::globaltimer();
        while (ptx::globaltimer() - t0 < 100000ull) {
        }
      } else if (*abort_flag) {
        // unwinding: give copies already in flight a bounded chance to land before the CTA leaves
        for (uint32_t k = (kbg > (uint32_t)STAGES ? kbg - STAGES : 0); k < kbg; ++k) {
          const unsigned long long t0 = ptx::globaltimer();
          while (!ptx::mbar_try_wait(&full[k % STAGES], (k / STAGES) & 1) && ptx::globaltimer() - t0 < 2000000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // The whole warp walks the loop and one elected lane issues: with warp-uniform control flow the descriptors
    // stay in uniform registers (under a branch on lane 0 each operand is moved there in front of every product).
    if (leader) {                                     // (the odd CTA's warp 1 only owns its tensor-memory allocation)
      uint32_t it = 0, s = 0, ph = 0;                 // ring position and its phase carry over tiles
      const uint32_t a_base = ptx::smem_u32(sA), b_base = ptx::smem_u32(sB);
      bool ok = true;
      for (uint32_t t = cta_first; t < total_tiles && ok; t += cta_step, ++it) {
        const uint32_t buf = it & 1, use = it >> 1;
        ok = __all_sync(0xFFFFFFFFu, ptx::mbar_wait(&tmem_empty[buf], (use & 1) ^ 1, abort_flag, g.status) ? 1 : 0) != 0;   // epilogue drained it
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * ACC_COLS;
        for (int kb = 0; kb < nkb; ++kb) {
          ok = __all_sync(0xFFFFFFFFu, ptx::mbar_wait(&full[s], ph, abort_flag, g.status) ? 1 : 0) != 0;
          if (!ok) break;
          ptx::tc_fence_after();
          // K-major, 128-byte swizzle: 8-row groups are 1024 bytes apart; one k16 step is 32 bytes
          // along the swizzled row.  MN-major: 64-row chunks are 8192 bytes apart (leading offset),
          // 8-deep k groups 1024 bytes apart, one k16 step is 2048 bytes.  A k16 step only moves the
          // start-address field of the descriptor, so the issuing thread adds a constant per MMA.
          const uint64_t ad0 = A_MN ? ptx::make_smem_desc(a_base + s * A_STAGE_BYTES, A_STAGE_BYTES / 2, 1024)
                                    : ptx::make_smem_desc(a_base + s * A_STAGE_BYTES, 16, 1024);
          const uint64_t bd0 = ptx::make_smem_desc(b_base + s * B_STAGE_BYTES, 16, 1024);
          constexpr uint64_t A_STEP = (A_MN ? 2048 : 32) >> 4, B_STEP = 32 >> 4;
          const bool last_kb = kb == nkb - 1;
          auto mma = [&](uint64_t ad, uint64_t bd, uint32_t acc) {
            if constexpr (PAIR) ptx::tc_mma_bf16_pair(d_tmem, ad, bd, IDESC, acc);
            else ptx::tc_mma_bf16(d_tmem, ad, bd, IDESC, acc);
          };
          if (ptx::elect_one()) {
            if (!last_kb || last_ksteps == BK / 16) {
              mma(ad0, bd0, kb ? 1u : 0u);
#pragma unroll
              for (int k = 1; k < BK / 16; ++k) mma(ad0 + k * A_STEP, bd0 + k * B_STEP, 1u);
            } else {
              for (int k = 0; k < last_ksteps; ++k) mma(ad0 + k * A_STEP, bd0 + k * B_STEP, (kb | k) ? 1u : 0u);
            }
            if constexpr (PAIR) {
              ptx::tc_commit_pair(&empty[s], 3);
              if (last_kb) ptx::tc_commit_pair(&tmem_full[buf], 3);
            } else {
              ptx::tc_commit(&empty[s]);
              if (last_kb) ptx::tc_commit(&tmem_full[buf]);
            }
          }
          __syncwarp();
          if (++s == STAGES) { s = 0; ph ^= 1; }
        }
      }
    }
  } else if (warp >= 2 + kEpiWarps) {
    // second producer: the B operand (long reductions only; a short one is
    // cheaper to feed from one thread)
    if (lane == 0 && two_producers) {
      uint32_t s = 0, ph = 1;
      bool ok = true;
      const uint32_t full0 = PAIR ? ptx::mapa(ptx::smem_u32(full), 0) : 0u;
      for (uint32_t t = cta_first; t < total_tiles && ok; t += cta_step) {
        const TileIdx ti_ = split_tile(t, g.fd_tiles_n, g.fd_tiles_m);
        const uint32_t tile_n = ti_.tile_n, batch = ti_.batch;
        const TileCoord tb = op_coords(g.cb, tile_n, batch, BN);
        const int brow0 = tb.row0 + (int)rank * BN_CTA;
        for (int kb = 0; kb < nkb; ++kb) {
          ok = ptx::mbar_wait(&empty[s], ph, abort_flag, g.status);
          if (!ok) break;
          if constexpr (PAIR) {
            if (leader) ptx::mbar_expect_tx(&full[s], 2 * B_STAGE_BYTES);
            tma_load_op_pair(g.cb, sB + s * B_STAGE_BYTES, &tmB, full0 + s * 8, kb * BK, brow0, tb);
          } else {
            ptx::mbar_expect_tx(&full[s], B_STAGE_BYTES);
            tma_load_op(g.cb, sB + s * B_STAGE_BYTES, &tmB, &full[s], kb * BK, tb.row0, tb);
          }
          if (++s == STAGES) { s = 0; ph ^= 1; }
        }
      }
    }
  } else {
    // Epilogue.  Warp (quadrant q, column group grp) owns rows q*32..q*32+31 (one TMEM lane per
    // thread) and CG = BN/4 columns, handled in rounds of RC <= 32 columns:
    //   phase 1 (thread = row): TMEM -> fp32 -> [RoPE] -> +bias -> [GELU] -> [+residual] -> bf16 -> staging row
    //   phase 2 (threads spread along the row): 16-byte stores, RC*2 contiguous bytes per row,
    // so a store instruction writes whole 32-byte sectors and several sectors of one line at once.
    constexpr int CG = BN / 4;
    constexpr bool DIRECT = PAIR;                            // rows leave the registers as 32-byte stores: no staging at all
    constexpr bool EARLY = DIRECT && LEAN;                   // accumulator slice to registers first, buffer released at once
    constexpr int RC = (BN == 256 && STAGES == 4 && !PAIR) ? 16 : (CG > 32 ? 32 : CG);   // 4 stages leave less staging room
    constexpr int ROUNDS = CG / RC;
    constexpr int RH = ROUNDS > 1 ? ROUNDS / 2 : 1;          // BN == 256: rounds [0, RH) hold the first halves of rotary pairs
    constexpr int VPR = RC / 8;                              // 16-byte vectors per row per round
    constexpr int STG_ROW = RC * 2 + 16;                     // bytes; the pad keeps phase 1 conflict-free
    const int e = warp - 2;
    const int q = warp & 3;                                  // TMEM lane quadrant this warp may read
    const int grp = e >> 2;
    constexpr bool QSTAGE = !DIRECT && !(BN == 256 && STAGES == 4);  // per-quadrant staging of whole rows
    constexpr bool QBULK = BN == 256 && !A_MN;               // staged rows leave as bulk copies (512-byte rows; not the MN-major-A kernel: 13.1 vs 12.1 us)
    constexpr int QROW = BN * 2 + 16;                        // bytes; the pad keeps phase 1 conflict-free
    uint8_t* stage = stage_base + e * (32 * STG_ROW);
    uint8_t* qstage = stage_base + q * (32 * QROW);
    uint32_t it = 0;
    bool ok = true;
    const bool res_wide = (reinterpret_cast<uintptr_t>(g.residual) & 31) == 0;   // (row offsets of a pair's output are multiples of 16 elements)
    constexpr bool PREFETCH_NEXT = false;                   // (tried: next-tile offset + residual a tile ahead; the extra live registers spill and it is slower)
    long long off_next = 0;
    uint4 res_next[VPR];
    const uint32_t tmem_empty0 = PAIR ? ptx::mapa(ptx::smem_u32(tmem_empty), 0) : 0u;   // the even CTA's barriers
    for (uint32_t t = cta_first; t < total_tiles && ok; t += cta_step, ++it) {
      const TileIdx ti_ = split_tile(t, g.fd_tiles_n, g.fd_tiles_m);
      const uint32_t tile_n = ti_.tile_n, tile_m = PAIR ? 2 * ti_.tile_m + rank : ti_.tile_m, batch = ti_.batch;
      const uint32_t buf = it & 1, use = it >> 1;
      const int n0 = tile_n * BN;
      const int row = tile_m * BM + q * 32 + lane;
      const bool row_ok = row < g.M;
      long long o2_base = 0;                                 // second copy: row = b * S + s goes to out2[b][col][s]
      if (!LEAN && g.out2) {
        const uint32_t b2 = fd_div((uint32_t)row, g.fd_out2_S);
        o2_base = (long long)b2 * g.N * g.fd_out2_S.d + ((uint32_t)row - b2 * g.fd_out2_S.d);
      }
      // Output offset of this thread's row (through the row map when the store is a scatter).  With
      // one round per tile the offset and the residual of the NEXT tile were requested during the
      // previous iteration, so neither the map evaluation nor the gather's latency is on the path
      // between the accumulator becoming ready and its buffer being handed back.
      // column-segmented output: a tile never straddles segments (seg_cols is a multiple of BN), so
      // the whole tile has one base and one pitch; the base is biased by the segment's first column
      __nv_bfloat16* out_t = g.out;
      long long ld_t = g.ldc;
      if (g.seg_cols > 0) {
        const int sg = n0 / g.seg_cols;
        out_t = g.seg_out[sg] - (long long)sg * g.seg_cols;
        ld_t = g.seg_ld[sg];
      }
      long long off;
      if (PREFETCH_NEXT && it > 0) {
        off = off_next;
      } else {
        off = 0;
        if (row_ok) off = g.has_rowmap ? devmap_eval_unrolled(g.rowmap, (uint32_t)row) : (long long)row * ld_t;
        off += (long long)batch * g.out_batch_stride;
      }
      const __nv_bfloat16* __restrict__ rrow = (!LEAN && g.residual) ? g.residual + off : nullptr;
      const bool rope_tile = !LEAN && (BN == 256 || BN == 128) && g.rope_cols > 0 && n0 < g.rope_cols;
      auto col_of = [&](int rd) {
        return BN == 256 ? 128 * (grp >> 1) + 32 * (grp & 1) + RC * (rd % RH) + 64 * (rd / RH) : grp * CG;
      };

      uint4 res[VPR];
      auto fetch_res = [&](int c0) {
        if constexpr (DIRECT) {                              // (pairs: full tiles, 32-byte aligned rows) whole sectors per load
          if (rrow && row_ok && res_wide) {
#pragma unroll
            for (int v = 0; v < VPR; v += 2) ptx::ld_global_v8(rrow + n0 + c0 + v * 8, res[v], res[v + 1]);
            return;
          }
        }
#pragma unroll
        for (int v = 0; v < VPR; ++v) {
          res[v] = make_uint4(0, 0, 0, 0);
          if (rrow && row_ok && n0 + c0 + v * 8 + 8 <= g.N) res[v] = *reinterpret_cast<const uint4*>(rrow + n0 + c0 + v * 8);
        }
      };
      if (PREFETCH_NEXT && it > 0) {
#pragma unroll
        for (int v = 0; v < VPR; ++v) res[v] = res_next[v];
      } else {
        fetch_res(col_of(0));                                // in flight while this tile's MMAs still run
      }
      if (PREFETCH_NEXT) {                                   // request the next tile's row offset and residual now
        const uint32_t tn = t + cta_step;
        if (tn < total_tiles) {
          const TileIdx nx = split_tile(tn, g.fd_tiles_n, g.fd_tiles_m);
          const int nrow = nx.tile_m * BM + q * 32 + lane;
          off_next = 0;
          if (nrow < g.M) off_next = g.has_rowmap ? devmap_eval_unrolled(g.rowmap, (uint32_t)nrow) : (long long)nrow * g.ldc;
          off_next += (long long)nx.batch * g.out_batch_stride;
          const int nn0 = nx.tile_n * BN, c0 = col_of(0);
#pragma unroll
          for (int v = 0; v < VPR; ++v) {
            res_next[v] = make_uint4(0, 0, 0, 0);
            if (g.residual && nrow < g.M && nn0 + c0 + v * 8 + 8 <= g.N)
              res_next[v] = *reinterpret_cast<const uint4*>(g.residual + off_next + nn0 + c0 + v * 8);
          }
        }
      }

      ok = ptx::mbar_wait(&tmem_full[buf], use & 1, abort_flag, g.status);
      if (!ok) break;
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + buf * ACC_COLS + ((uint32_t)(q * 32) << 16);
      if constexpr (QSTAGE && QBULK) {
        // the previous tile's row copies have read the staging rows before anyone overwrites them
        if (lane < 8) ptx::bulk_wait_group_read<0>();
        asm volatile("bar.sync %0, 128;" ::"r"(1 + q) : "memory");
      }

      // EARLY: the whole accumulator slice of the thread (ROUNDS x RC values) moves to registers first and the buffer goes
      // back to the issuing warp before any arithmetic or store, so the next tile but one starts as early as it can
      uint32_t rall[EARLY ? ROUNDS : 1][RC];
      if constexpr (EARLY) {
#pragma unroll
        for (int rd = 0; rd < ROUNDS; ++rd) ptx::tmem_ld_cols<RC>(taddr + col_of(rd), rall[rd]);
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_cluster(tmem_empty0 + buf * 8);
      }
#pragma unroll
      for (int rd = 0; rd < ROUNDS; ++rd) {
        const int c0 = col_of(rd);
        float acc[RC];
        uint4 bv[VPR];                                       // this round's bias columns: requested before the wait on tensor memory
        if (g.bias) {
#pragma unroll
          for (int v = 0; v < VPR; ++v) {
            bv[v] = make_uint4(0, 0, 0, 0);
            if (n0 + c0 + v * 8 + 8 <= g.N) bv[v] = *reinterpret_cast<const uint4*>(g.bias + n0 + c0 + v * 8);
          }
        }
        {
          uint32_t rv_local[EARLY ? 1 : RC], rw[EARLY ? 1 : RC];
          uint32_t* rv = EARLY ? rall[EARLY ? rd : 0] : rv_local;
          if constexpr (!EARLY) ptx::tmem_ld_cols<RC>(taddr + c0, rv);
          // rotary pairs are (i, i + R/2) inside the first R columns of a 128-column head (R = 128: the
          // whole head).  This round's RC columns start at head-local column hc0; they rotate iff hc0 < R,
          // and their partners are the RC columns R/2 further up or down (or, when R/2 < RC, the other
          // half of this very round), read from TMEM a second time.
          const int hc0 = c0 & 127, half = g.rope_half;
          if (rope_tile && hc0 < 2 * half) {
            const bool in_round = half < RC;                 // R = 32 with 32-column rounds: pairs (j, j + 16) of this round
            const bool first_half = hc0 < half;
            if constexpr (!EARLY) {
              if (!in_round) ptx::tmem_ld_cols<RC>(taddr + (first_half ? c0 + half : c0 - half), rw);
              ptx::tmem_ld_wait();
            }
            // angle = position * theta^(-i/(R/2)), reduced mod 2 pi in two steps, then the hardware
            // sine / cosine: no table traffic (a [S, 64] table read 16 bytes per lane per row
            // slowed the whole kernel by a fifth)
            const float pos = (float)(row_ok ? g.rope_pos0 + row % g.rope_S : 0);
            const int i0 = in_round ? 0 : hc0 - (first_half ? 0 : half);
#pragma unroll
            for (int j = 0; j < RC; ++j) {
              const bool fh = in_round ? j < RC / 2 : first_half;
              const int i = in_round ? (j & (RC / 2 - 1)) : i0 + j;
              float f;
              asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(f) : "f"(-(float)i * g.rope_c));
              const float ang = pos * f;
              const float kk = rintf(ang * 0.15915494309189535f);
              float red = fmaf(-kk, 6.2831854820251465f, ang);
              red = fmaf(kk, 1.7484556e-7f, red);
              const float sn = __sinf(red), cs = __cosf(red);
              const float x = __uint_as_float(rv[j]);
              const float y = __uint_as_float(in_round ? rv[j ^ (RC / 2)] : rw[j]);
              acc[j] = fh ? x * cs - y * sn : x * cs + y * sn;
            }
          } else {
            if constexpr (!EARLY) ptx::tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < RC; ++j) acc[j] = __uint_as_float(rv[j]);
          }
        }
        if (g.bias) {
#pragma unroll
          for (int v = 0; v < VPR; ++v) {
            const uint32_t w[4] = {bv[v].x, bv[v].y, bv[v].z, bv[v].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float2 f = bf16x2_to_float2(w[j]);
              acc[v * 8 + 2 * j] += f.x;
              acc[v * 8 + 2 * j + 1] += f.y;
            }
          }
        }
        if (g.gelu) {
#pragma unroll
          for (int j = 0; j < RC; ++j) acc[j] = gelu_fast(acc[j]);
        }
        if (rrow) {
#pragma unroll
          for (int v = 0; v < VPR; ++v) {
            const uint32_t w[4] = {res[v].x, res[v].y, res[v].z, res[v].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float2 f = bf16x2_to_float2(w[j]);
              acc[v * 8 + 2 * j] += f.x;
              acc[v * 8 + 2 * j + 1] += f.y;
            }
          }
          if (rd + 1 < ROUNDS) fetch_res(col_of(rd + 1));
        }
        if (!LEAN && g.out2 && row_ok) {
          // The redundant copy of a producer with consumers of different reduction dimensions: the same values with the
          // row's position inside its group as the contiguous dimension.  A warp's 32 rows write 64 contiguous bytes per column.
#pragma unroll
          for (int j = 0; j < RC; ++j)
            if (n0 + c0 + j < g.N) g.out2[o2_base + (long long)(n0 + c0 + j) * g.fd_out2_S.d] = __float2bfloat16_rn(acc[j]);
        }
        uint4 pk_prev = make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int v = 0; v < VPR; ++v) {
          uint4 pk;
          pk.x = float2_to_bf16x2(acc[v * 8 + 0], acc[v * 8 + 1]);
          pk.y = float2_to_bf16x2(acc[v * 8 + 2], acc[v * 8 + 3]);
          pk.z = float2_to_bf16x2(acc[v * 8 + 4], acc[v * 8 + 5]);
          pk.w = float2_to_bf16x2(acc[v * 8 + 6], acc[v * 8 + 7]);
          if constexpr (DIRECT) {
            // 64 contiguous bytes of the thread's own row per round, as two 32-byte stores: whole sectors, and the
            // shared memory (whose bandwidth the operands need) is left to the ring, which gets six stages
            if (LEAN && g.tma_out) {
              // lean epilogue: the warp's 32 x 32 box goes through its own 2 KB of shared memory and leaves as one TMA
              // store -- a row-per-thread store touches 32 lines per instruction, and those stores and the next tile's
              // operand loads were in each other's way
              if (v == 0) {
                if (lane == 0) ptx::bulk_wait_group_read<0>();     // the previous round's box has been read
                __syncwarp();
              }
              *reinterpret_cast<uint4*>(cstage + e * CBOX_BYTES + lane * 64 + ((v ^ ((lane >> 1) & 3)) << 4)) = pk;
              if (v == VPR - 1) {
                ptx::fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                  ptx::tma_store_2d(&tmC, cstage + e * CBOX_BYTES, n0 + c0, (int)tile_m * BM + q * 32);
                  ptx::bulk_commit_group();
                }
              }
            } else if (v & 1) {
              if (row_ok) ptx::st_global_v8(out_t + off + n0 + c0 + (v - 1) * 8, pk_prev, pk);
            } else {
              pk_prev = pk;
            }
          } else if constexpr (QSTAGE) *reinterpret_cast<uint4*>(qstage + lane * QROW + (c0 + v * 8) * 2) = pk;
          else *reinterpret_cast<uint4*>(stage + lane * STG_ROW + v * 16) = pk;
        }
        if constexpr (!QSTAGE && !DIRECT) {
          __syncwarp();
#pragma unroll
          for (int i = 0; i < VPR; ++i) {
            const int v = lane + 32 * i;
            const int rr = v / VPR, seg = v - rr * VPR;
            const long long roff = __shfl_sync(0xFFFFFFFFu, off, rr);
            const int rok = __shfl_sync(0xFFFFFFFFu, (int)row_ok, rr);
            const uint4 pk = *reinterpret_cast<const uint4*>(stage + rr * STG_ROW + seg * 16);
            if (rok && n0 + c0 + seg * 8 + 8 <= g.N) *reinterpret_cast<uint4*>(out_t + roff + n0 + c0 + seg * 8) = pk;
          }
          __syncwarp();
        }
      }
      // all of this warp's TMEM reads of the buffer have completed (wait::ld above)
      if constexpr (!EARLY) {
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if constexpr (PAIR) ptx::mbar_arrive_cluster(tmem_empty0 + buf * 8);
          else ptx::mbar_arrive(&tmem_empty[buf]);
        }
      }
      if constexpr (QSTAGE && QBULK) {
        // the four warps of the quadrant have filled a 32 x 256 staging tile: every 512-byte row leaves as one bulk copy
        // (shared memory -> global), eight rows per warp, so no thread spends instructions on moving the tile.  Measured:
        // the batched q k^T GEMM 78.4 -> 72.6 us; on 192-byte rows (the 96-wide scatter GEMM) the same was slower, 22.3 vs
        // 20.7 us, so narrower tiles keep the vector loop below.
        ptx::fence_proxy_async();
        asm volatile("bar.sync %0, 128;" ::"r"(1 + q) : "memory");
        const int rr = grp * 8 + (lane & 7);
        const long long roff = __shfl_sync(0xFFFFFFFFu, off, rr);
        const int rok = __shfl_sync(0xFFFFFFFFu, (int)row_ok, rr);
        const int ncols = g.N - n0 < BN ? g.N - n0 : BN;
        if (lane < 8) {
          if (rok) ptx::bulk_store(out_t + roff + n0, qstage + rr * QROW, (uint32_t)ncols * 2u);
          ptx::bulk_commit_group();
        }
      } else if constexpr (QSTAGE) {
        // the four warps of the quadrant have filled a 32 x BN staging tile: store whole rows
        constexpr int VR = BN / 8;                           // 16-byte vectors per row
        asm volatile("bar.sync %0, 128;" ::"r"(1 + q) : "memory");
        const int tq = grp * 32 + lane;
#pragma unroll
        for (int i = 0; i < VR / 4; ++i) {
          const int v = tq + 128 * i;
          const int rr = v / VR, seg = v - rr * VR;
          const long long roff = __shfl_sync(0xFFFFFFFFu, off, rr);
          const int rok = __shfl_sync(0xFFFFFFFFu, (int)row_ok, rr);
          const uint4 pk = *reinterpret_cast<const uint4*>(qstage + rr * QROW + seg * 16);
          if (rok && n0 + seg * 8 + 8 <= g.N) *reinterpret_cast<uint4*>(out_t + roff + n0 + seg * 8) = pk;
        }
        asm volatile("bar.sync %0, 128;" ::"r"(1 + q) : "memory");
      }
    }
  }
  ptx::bulk_wait_group_read<0>();   // output boxes of the last tile have been read out of shared memory
  ptx::tc_fence_before();
  if constexpr (PAIR) {
    __syncwarp();
    ptx::cluster_sync();            // neither CTA leaves (or frees tensor memory) while the other may still read or signal it
  } else {
    __syncthreads();
  }
  if (warp == 1) {
    ptx::tc_fence_after();
    if constexpr (PAIR) ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
    else ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------------
// Host side: tensor maps.
// ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

std::mutex g_tm_mu;
std::unordered_map<std::string, CUtensorMap> g_tm_cache;

int encode_cached(const void* ptr, int rank, const uint64_t* dims, const uint64_t* strides_b, const uint32_t* box,
                  CUtensorMap* out, int swizzle_bytes = 128) {
  std::string key((const char*)&ptr, sizeof(ptr));
  key.append((const char*)&rank, sizeof(rank));
  key.append((const char*)dims, sizeof(uint64_t) * rank);
  key.append((const char*)strides_b, sizeof(uint64_t) * (rank - 1));
  key.append((const char*)box, sizeof(uint32_t) * rank);
  key.append((const char*)&swizzle_bytes, sizeof(int));
  {
    std::lock_guard<std::mutex> lk(g_tm_mu);
    auto it = g_tm_cache.find(key);
    if (it != g_tm_cache.end()) {
      *out = it->second;
      return SMARTMEM_OK;
    }
  }
  EncodeTiledFn enc = get_encode();
  if (!enc) return SMARTMEM_ERR_CUDA;
  cuuint64_t d[5], s[4];
  cuuint32_t b[5], es[5];
  for (int i = 0; i < rank; ++i) {
    d[i] = dims[i];
    b[i] = box[i];
    es[i] = 1;
    if (i < rank - 1) s[i] = strides_b[i];
  }
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(ptr), d, s, b, es,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return SMARTMEM_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_tm_mu);
  if (g_tm_cache.size() > 4096) g_tm_cache.clear();
  g_tm_cache[key] = *out;
  return SMARTMEM_OK;
}

// Turns an operand description into a tensor map + the coordinate rule of the kernel.
// `box_rows` rows per copy (a CTA pair fetches a tile of `tile_rows` rows as two boxes, one per CTA).
int build_operand(const TcOperand& op, int tile_rows, int box_rows, CUtensorMap* tm, OpCoord* oc) {
  if (op.n_row_atoms < 1 || op.n_row_atoms + op.n_batch_atoms > 4) return SMARTMEM_ERR_UNSUPPORTED;
  if (((uintptr_t)op.ptr & 15) != 0) return SMARTMEM_ERR_ALIGNMENT;
  const int nr = op.n_row_atoms, nb = op.n_batch_atoms;
  const long long in_ext = op.row_extent[nr - 1], in_str = op.row_stride[nr - 1];
  const bool mn = op.k_stride != 1;
  if (mn && in_str != 1) return SMARTMEM_ERR_UNSUPPORTED;
  if (nr > 1 && in_ext % tile_rows) return SMARTMEM_ERR_UNSUPPORTED;
  uint64_t dims[5], strides[4];
  uint32_t box[5];
  int rank = 0;
  auto push = [&](long long ext, long long str_elems, uint32_t bx) -> bool {
    if (rank > 0) {
      if ((str_elems * 2) % 16 || str_elems <= 0) return false;
      strides[rank - 1] = (uint64_t)str_elems * 2;
    }
    dims[rank] = (uint64_t)ext;
    box[rank] = bx;
    ++rank;
    return true;
  };
  bool ok = true;
  if (!mn) {
    ok = ok && push(op.K, 1, BK) && push(in_ext, in_str, (uint32_t)box_rows);
  } else {
    ok = ok && push(in_ext, 1, 64) && push(op.K, op.k_stride, BK);
  }
  memset(oc, 0, sizeof(*oc));
  for (int i = nr - 2; i >= 0 && ok; --i) {
    ok = push(op.row_extent[i], op.row_stride[i], 1);
    oc->outer[oc->n_outer++] = make_fastdiv((uint32_t)op.row_extent[i]);
    oc->n_outer_row++;
  }
  for (int i = nb - 1; i >= 0 && ok; --i) {
    ok = push(op.batch_extent[i], op.batch_stride[i], 1);
    oc->outer[oc->n_outer++] = make_fastdiv((uint32_t)op.batch_extent[i]);
  }
  if (!ok) return SMARTMEM_ERR_UNSUPPORTED;
  if (rank < 2) return SMARTMEM_ERR_UNSUPPORTED;
  while (rank < 5) {                                   // pad: all kernels issue 5-D loads
    strides[rank - 1] = strides[rank - 2] * dims[rank - 1];
    if (strides[rank - 1] >= (1ull << 40)) strides[rank - 1] = strides[rank - 2];
    dims[rank] = 1;
    box[rank] = 1;
    ++rank;
  }
  oc->rank = rank;
  oc->mn_major = mn ? 1 : 0;
  oc->tiles_inner = make_fastdiv((uint32_t)((in_ext + tile_rows - 1) / tile_rows));
  return encode_cached(op.ptr, rank, dims, strides, box, tm);
}

// every offset the map can produce is a multiple of `q` elements
bool devmap_offsets_multiple_of(const DevMap& m, long long q) {
  if (m.base % q) return false;
  for (int a = 0; a < m.n_atoms; ++a)
    if (m.roll_of[a] < 0 && m.stride[a] % q) return false;
  for (int r = 0; r < m.n_rolls; ++r) {
    if (m.roll_stride[r] % q) return false;
    for (int i = 0; i < m.roll_n_parts[r] && m.roll_n_parts[r] > 1; ++i)
      if (m.roll_part_stride[r][i] % q) return false;
  }
  return true;
}

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
  }
  return n;
}

template <int BN, int STAGES, bool A_MN, bool PAIR = false, bool LEAN = false>
int launch_t(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, const GemmArgs& g, cudaStream_t st) {
  constexpr bool QST = !PAIR && !(BN == 256 && STAGES == 4);
  constexpr int RCc = !QST ? 16 : ((BN / 4) > 32 ? 32 : (BN / 4));
  constexpr size_t smem = 1024 + STAGES * (A_STAGE_BYTES + (PAIR ? BN / 2 : BN) * BK * 2) + (2 * STAGES + 4) * 8 + 16 +
                          (LEAN ? kEpiWarps * 32 * 64 : PAIR ? 0 : !QST ? kEpiWarps * 32 * (RCc * 2 + 16) : 4 * 32 * (BN * 2 + 16));   // pairs store from registers
  if (ensure_max_dynamic_smem((const void*)gemm_tc_kernel<BN, STAGES, A_MN, PAIR, LEAN>, (int)smem) != SMARTMEM_OK) return SMARTMEM_ERR_CUDA;
  profile_tick("gemm_tc", st);
  const long long tiles = (long long)g.tiles_n * g.tiles_m * g.batch;
  if constexpr (PAIR) {
    // one cluster of two CTAs per tile of 256 rows; the two CTAs of a cluster are neighbours in blockIdx.x
    const long long pairs = sm_count() / 2;
    const unsigned grid = (unsigned)(2 * (tiles < pairs ? tiles : pairs));
    launch_pdl_cluster(gemm_tc_kernel<BN, STAGES, A_MN, PAIR, LEAN>, dim3(grid), dim3(kThreads), smem, st, 2u, ta, tb, tc, g);
  } else {
    const unsigned grid = (unsigned)(tiles < sm_count() ? tiles : sm_count());
    launch_pdl(gemm_tc_kernel<BN, STAGES, A_MN, PAIR, LEAN>, dim3(grid), dim3(kThreads), smem, st, ta, tb, tc, g);
  }
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

}  // namespace

int tc_encode_2d(const void* ptr, long long inner, long long outer, long long pitch_elems, int box_inner, int box_outer,
                 CUtensorMap* out) {
  if (((uintptr_t)ptr & 15) || (pitch_elems * 2) % 16) return SMARTMEM_ERR_ALIGNMENT;
  const uint64_t dims[2] = {(uint64_t)inner, (uint64_t)outer};
  const uint64_t strides[1] = {(uint64_t)pitch_elems * 2};
  const uint32_t box[2] = {(uint32_t)box_inner, (uint32_t)box_outer};
  return encode_cached(ptr, 2, dims, strides, box, out);
}

int tc_encode_2d_sw64(const void* ptr, long long inner, long long outer, long long pitch_elems, int box_inner,
                      int box_outer, CUtensorMap* out) {
  if (((uintptr_t)ptr & 15) || (pitch_elems * 2) % 16 || box_inner * 2 != 64) return SMARTMEM_ERR_ALIGNMENT;
  const uint64_t dims[2] = {(uint64_t)inner, (uint64_t)outer};
  const uint64_t strides[1] = {(uint64_t)pitch_elems * 2};
  const uint32_t box[2] = {(uint32_t)box_inner, (uint32_t)box_outer};
  return encode_cached(ptr, 2, dims, strides, box, out, 64);
}

int tc_encode_nd_sw64(const void* ptr, int rank, const long long* dims, const long long* strides_elems, const int* box,
                      CUtensorMap* out) {
  if (rank < 2 || rank > 5 || ((uintptr_t)ptr & 15) || box[0] * 2 != 64) return SMARTMEM_ERR_ALIGNMENT;
  uint64_t d[5], sb[4];
  uint32_t b[5];
  for (int i = 0; i < rank; ++i) {
    d[i] = (uint64_t)dims[i];
    b[i] = (uint32_t)box[i];
    if (i > 0) {
      sb[i - 1] = (uint64_t)strides_elems[i - 1] * 2;
      if (sb[i - 1] % 16) return SMARTMEM_ERR_ALIGNMENT;
    }
  }
  return encode_cached(ptr, rank, d, sb, b, out, 64);
}

int tc_sm_count() { return sm_count(); }

int tc_operand_from_map(const smartmem_index_map_t& m, int n_batch_atoms, int n_row_atoms, const void* ptr,
                        TcOperand* op) {
  if (m.klass == 3 || m.n_rolls > 0) return SMARTMEM_ERR_UNSUPPORTED;
  const int nk = m.n_atoms - n_batch_atoms - n_row_atoms;
  if (nk != 1 || n_row_atoms < 1 || n_row_atoms > 3 || n_batch_atoms > 3) return SMARTMEM_ERR_UNSUPPORTED;
  memset(op, 0, sizeof(*op));
  op->ptr = (const char*)ptr + m.base * 2;
  op->n_batch_atoms = n_batch_atoms;
  op->n_row_atoms = n_row_atoms;
  for (int i = 0; i < n_batch_atoms; ++i) {
    op->batch_extent[i] = m.extent[i];
    op->batch_stride[i] = m.src_stride[i];
  }
  for (int i = 0; i < n_row_atoms; ++i) {
    op->row_extent[i] = m.extent[n_batch_atoms + i];
    op->row_stride[i] = m.src_stride[n_batch_atoms + i];
  }
  op->K = m.extent[m.n_atoms - 1];
  op->k_stride = m.src_stride[m.n_atoms - 1];
  return SMARTMEM_OK;
}

TcOperand tc_operand_plain(const void* ptr, long long rows, long long K, long long ld) {
  TcOperand op;
  memset(&op, 0, sizeof(op));
  op.ptr = ptr;
  op.n_row_atoms = 1;
  op.row_extent[0] = rows;
  op.row_stride[0] = ld;
  op.K = K;
  op.k_stride = 1;
  return op;
}

int launch_gemm_tc(const TcOperand& A, const TcOperand& B, const TcEpilogue& ep, long long batch, long long M,
                   long long N, long long K, cudaStream_t st) {
  if (M < 1 || N < 1 || K < 1 || batch < 1 ||  M >= (1ll << 31) || N >= (1ll << 31))
    return SMARTMEM_ERR_UNSUPPORTED;
  if (A.K != K || B.K != K) return SMARTMEM_ERR_SHAPE;
  if (((uintptr_t)ep.out & 15) || ((uintptr_t)ep.residual & 15) || ((uintptr_t)ep.bias & 15) || ep.ldc % 8 ||
      ep.out_batch_stride % 8)
    return SMARTMEM_ERR_ALIGNMENT;
  if (N % 8) return SMARTMEM_ERR_UNSUPPORTED;
  const bool a_mn = A.k_stride != 1;
  if (B.k_stride != 1) return SMARTMEM_ERR_UNSUPPORTED;
  // tile width: the widest of {256, 128, 96, 64} that divides N (fewest wasted columns), else 128
  int bn = 128;
  if (ep.rope_cols > 0) bn = (M <= BM && batch == 1 && N / 256 < tc_sm_count()) ? 128 : 256;   // one head or two per tile
  else if (N % 256 == 0) {
    // 256 or 128 wide: whichever leaves fewer idle SMs in the last wave (time of a wave ~ tile width plus a fixed part).
    // Only for short reductions: a 128-wide tile reads as many operand bytes per product as shared memory delivers,
    // so over a long K the wider tile wins even with a ragged last wave (measured at K = 2048).
    const long long tm = (M + BM - 1) / BM * batch, sms = tc_sm_count();
    const long long w256 = (tm * (N / 256) + sms - 1) / sms, w128 = (tm * (N / 128) + sms - 1) / sms;
    bn = (K <= 1024 && w128 * (128 + 48) < w256 * (256 + 48)) ? 128 : 256;
  } else if (N % 128 == 0) bn = 128;
  else if (N % 96 == 0) bn = 96;
  else if (N % 64 == 0) bn = 64;
  // One row tile only (a decode step: M <= 128) and few wide column tiles: the GEMM streams the weight
  // once and is bound by how many SMs pull on it, so take the narrowest tile that divides N.
  if (ep.rope_cols == 0 && batch == 1 && M <= BM && !a_mn && N % 64 == 0 && N / bn < tc_sm_count()) bn = 64;
  if (a_mn && bn < 128) bn = 128;                         // MN-major A operands come with 128- and 256-wide tiles only
  if (ep.rope_cols > 0 && (N % 256 || ep.rope_cols % 256 || ep.rope_S < 1)) return SMARTMEM_ERR_UNSUPPORTED;
  if (ep.rope_cols > 0 && ep.rope_dim != 0 && ep.rope_dim != 32 && ep.rope_dim != 64 && ep.rope_dim != 128) return SMARTMEM_ERR_UNSUPPORTED;
  if (ep.seg_cols > 0) {
    if (ep.seg_cols % 256 || N > 3ll * ep.seg_cols || ep.rowmap || ep.residual || batch != 1) return SMARTMEM_ERR_UNSUPPORTED;
    for (int i = 0; i * (long long)ep.seg_cols < N; ++i)
      if (!ep.seg_out[i] || ((uintptr_t)ep.seg_out[i] & 15) || ep.seg_ld[i] % 8) return SMARTMEM_ERR_ALIGNMENT;
  }
  const int nkb = (int)((K + BK - 1) / BK);
  // 256 wide, short K: wider store rounds instead of a 4th stage.  Narrow tiles: their stages are
  // small, and a tile is consumed faster than a load's latency, so the ring runs several tiles ahead.
  const int stages = bn == 256 ? (nkb <= 4 ? 3 : 4) : (bn <= 96 ? 6 : 4);
  // CTA pairs (two SMs on one 256 x 256 tile) where the row tiles pair up and there is more than one wave of work for
  // the single-CTA kernel: below that the operand feed is not what bounds the GEMM.
  // SMARTMEM_GEMM_PAIR=0 keeps every GEMM on single CTAs (for measuring what pairing buys).
  static const int allow_pair = [] { const char* e = getenv("SMARTMEM_GEMM_PAIR"); return (e && e[0] == '0') ? 0 : 1; }();
  const long long tiles_m1 = (M + BM - 1) / BM;
  const bool pair = allow_pair && (bn == 256 || bn == 128) && !a_mn && tiles_m1 % 2 == 0 && nkb > 4 && N % 256 == 0 &&
              tiles_m1 * (N / 256) * batch > tc_sm_count() &&
              (!ep.rowmap || devmap_offsets_multiple_of(*ep.rowmap, 16)) && ep.seg_cols == 0 && !ep.out2 && ep.ldc % 16 == 0 &&
              ep.out_batch_stride % 16 == 0 && ((uintptr_t)ep.out & 31) == 0;   // (its epilogue writes 32-byte vectors)
  if (pair) {
    // width of a pair's tile: 256 unless the last wave of 256-wide tiles is so ragged that the waves of half the width
    // are shorter.  Microseconds per tile, fitted to measurements: per k-block a 256-wide tile costs its products and a
    // 128-wide one its operand feed (about 2/3 of that), plus a fixed part for the epilogue the ring cannot hide.
    const long long pairs = tc_sm_count() / 2, t256 = tiles_m1 / 2 * (N / 256) * batch;
    const long long w256 = (t256 + pairs - 1) / pairs, w128 = (2 * t256 + pairs - 1) / pairs;
    bn = (ep.rope_cols == 0 && w128 * (nkb * 0.21 + 1.2) < w256 * (nkb * 0.33 + 2.2)) ? 128 : 256;
  }
  GemmArgs g;
  memset(&g, 0, sizeof(g));
  CUtensorMap ta, tb;
  int rc = build_operand(A, BM, BM, &ta, &g.ca);
  if (rc != SMARTMEM_OK) return rc;
  rc = build_operand(B, bn, pair ? bn / 2 : bn, &tb, &g.cb);
  if (rc != SMARTMEM_OK) return rc;
  g.M = (int)M; g.N = (int)N; g.K = (int)K;
  g.out = (__nv_bfloat16*)ep.out;
  g.ldc = ep.ldc;
  g.out_batch_stride = ep.out_batch_stride;
  g.bias = (const __nv_bfloat16*)ep.bias;
  g.residual = (const __nv_bfloat16*)ep.residual;
  g.gelu = ep.gelu;
  g.has_rowmap = ep.rowmap ? 1 : 0;
  if (ep.rowmap) g.rowmap = *ep.rowmap;
  g.rope_cols = ep.rope_cols;
  g.rope_S = ep.rope_S;
  g.rope_pos0 = ep.rope_pos0;
  g.seg_cols = ep.seg_cols;
  for (int i = 0; i < 3; ++i) { g.seg_out[i] = (__nv_bfloat16*)ep.seg_out[i]; g.seg_ld[i] = ep.seg_ld[i]; }
  const int rope_dim = ep.rope_dim ? ep.rope_dim : 128;
  g.rope_half = rope_dim / 2;
  g.rope_c = ep.rope_log2_theta / (float)(rope_dim / 2);
  if (ep.out2) {
    if (ep.out2_S < 1 || M % ep.out2_S || batch != 1 || ((uintptr_t)ep.out2 & 1)) return SMARTMEM_ERR_UNSUPPORTED;
    g.out2 = (__nv_bfloat16*)ep.out2;
    g.fd_out2_S = make_fastdiv((uint32_t)ep.out2_S);
  }
  g.status = device_status_ptr();
  if (!g.status) return SMARTMEM_ERR_CUDA;
  g.tiles_n = (int)((N + bn - 1) / bn);
  g.tiles_m = (int)(pair ? tiles_m1 / 2 : tiles_m1);       // pairs walk over tiles of 256 rows
  g.fd_tiles_n = make_fastdiv((uint32_t)g.tiles_n);
  g.fd_tiles_m = make_fastdiv((uint32_t)g.tiles_m);
  g.batch = (int)batch;
  if ((long long)g.tiles_n * g.tiles_m * g.batch >= (1ll << 31)) return SMARTMEM_ERR_UNSUPPORTED;
  CUtensorMap tc = ta;                                     // (a valid map for the kernels that store without TMA)
  if (pair && bn == 256 && nkb <= 16 && ep.rope_cols == 0 && !ep.residual) {
    if (batch == 1 && !ep.rowmap) {                        // output as 32 x 32 boxes of [M, N] with pitch ldc
      const uint64_t dims[2] = {(uint64_t)N, (uint64_t)M}, strides[1] = {(uint64_t)ep.ldc * 2};
      const uint32_t box[2] = {32, 32};
      if (encode_cached(ep.out, 2, dims, strides, box, &tc, 64) == SMARTMEM_OK) g.tma_out = 1;
      else tc = ta;
    }
    return launch_t<256, 6, false, true, true>(ta, tb, tc, g, st);
  }
  if (pair && bn == 256) return launch_t<256, 6, false, true>(ta, tb, tc, g, st);
  if (pair) return launch_t<128, 8, false, true>(ta, tb, tc, g, st);
#define SM_CASE(BN_, ST_, MN_)                                                                  \
  if (bn == BN_ && stages == ST_ && a_mn == MN_) return launch_t<BN_, ST_, MN_>(ta, tb, tc, g, st);
  SM_CASE(256, 3, false) SM_CASE(256, 4, false) SM_CASE(128, 4, false) SM_CASE(96, 6, false) SM_CASE(64, 6, false)
  SM_CASE(256, 3, true) SM_CASE(256, 4, true) SM_CASE(128, 4, true)
#undef SM_CASE
  return SMARTMEM_ERR_UNSUPPORTED;
}

}  // namespace smartmem
