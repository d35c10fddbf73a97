// Attention half of a narrow Swin block (head dimension 32, 2 or 3 heads, C = 32 * heads) in ONE kernel:
//
//   y = x + unshift(unpartition( proj( window_attention( qkv( LN1( partition(shift(x)) ) ) ) ) ))
//
// The cyclic shift, the window partition, the head split, the K transpose, the head merge, the window
// reverse and the reverse shift are all index arithmetic here: rows of x are gathered through the
// composed shift o partition map straight into the MMA operand layout, q / k / v and the attention
// output never leave the SM, and the result rows are scattered through the same map.  Per token the
// kernel reads C and writes C elements of global memory; the three-kernel form of the same chain
// moves 11 C through HBM.
//
// Unit of work: a pair of windows = one 128-row MMA tile (window w of the pair in rows 64 w .. 64 w + T - 1,
// the rows between T and 64 stay zero), taken round-robin by persistent CTAs that keep every weight resident.
// An "item" is (unit, head); head h is the work of row group h.  Per item, all in one 96-column buffer of tensor
// memory (four buffers in rotation):
//
//   acc  = [X | e] [Wq_h; Wk_h; Wv_h | f]^T    128 x 96 x (C + 16)  tcgen05; X = the RAW rows (bf16) in shared memory
//   q,k,v = rstd acc                           LayerNorm applied algebraically (below); q goes back to tensor memory as
//                                              bf16 pairs, k and v to shared memory in operand layout
//   S    = [q0 0; 0 q1] [k0 | k1]^T            128 x 64 x 64: the two windows' keys are stacked along the reduction
//                                              dimension and each query row carries zeros in the other window's half,
//                                              so a row's 64 scores are its own window's; q is read from tensor memory
//   P    = softmax(scale S + bias + mask)      one query row per thread (= its TMEM lane); P stored as bf16 pairs
//   O    = [P0 0; 0 P1] [v0; v1]               128 x 32 x 128, P read from tensor memory, V as it lies (MN-major)
//   Ob   = bf16(O / rowsum)                    back into tensor memory as packed pairs
//   Y   += Ob Wp[:, 32 h : 32 h + 32]^T        128 x C x 32: the head merge is the accumulation over heads
//
// and per unit  Y starts as X I (the unit's raw rows times the identity: the residual rides on the tensor core, exactly, since
// every product is a bf16 value times one), the heads' projections accumulate on top, and the epilogue stores
// y_row = Y + b_proj with 16-byte vectors at the row's offset under the map.
//
// LayerNorm without a normalised tile:  LN(x) W^T + b = rstd (x W'^T - mean c + sigma b'),  W' = bf16(gamma . W) (column
// scaling), c_n = sum_k W'_nk, b'_n = b_n + sum_k beta_k W_nk, sigma = 1 / rstd.  c is summed from the ROUNDED W', so the
// mean term cancels exactly what the raw rows contribute through W' -- rows with a large common offset lose nothing.  The two
// rank-one terms ride on the tensor core as one extra k-step: row r of the operand carries (-mean_r, sigma_r), column n of the
// weights (c_n, b'_n), each fp32 value split into three bf16 pieces (the six largest cross products of the pieces are kept:
// exact to 2^-24), so the epilogue of the QKV product is one multiply per element.  Every CTA folds gamma into its resident
// copy of the weights once (prologue); the row statistics are two passes over the row, fp32.
//
// Warp roles (9 + 4 heads warps):
//   0-3   bring in the rows of the units ahead -- a window that does not straddle the seam of the shifted image is an affine
//         box [32 channels, ws, ws] of x per k-block, one TMA copy each; a seam window is gathered row by row with 16-byte
//         asynchronous copies through the index map -- and take their statistics, a thread per row;
//   then  one group of four warps per head (q/k/v epilogue, softmax, O epilogue: one row of the pair tile per thread).  A
//         group issues its own S and P V products from an elected thread right after the group's barrier: those hand-offs
//         are on the item's critical path, and a barrier is cheaper than a trip through another warp;
//   then  four warps for the Y epilogue (one row per thread);
//   last  one thread that issues, in item order, the products that have slack: QKV of the items ahead (into the buffer the
//         item four before has left), the residual product that opens a unit's Y, and the heads' projections.  Issue order is
//         accumulation order, and orders a buffer's next accumulator behind the projection that reads the buffer last.
// What bounds it (clock stamps at every hand-off, and builds with the arithmetic of one role removed): not arithmetic -- with
// the whole softmax compiled out the kernel is 5 % faster -- but the chain of hand-offs of an item (tensor-memory round trips,
// three barriers, two waits for small products behind other groups' products in the tensor pipe), about 9000 cycles per item
// with three items in flight; and instruction fetch: code that runs once per unit (statistics, epilogue, the prologue) is
// kept in rolled loops because its straight-line form ran at the speed of the instruction cache misses.  Every wait is bounded.
#include "attn.cuh"
#include "gemm_tc.cuh"
#include "ptx.cuh"
#include "tc_tiles.cuh"


namespace smartmem {
namespace {

using ptx::f32x2;

#define GWAIT(bar, par) ptx::mbar_wait(bar, par, abort_flag, g.status)

constexpr int D = 32, TP = 64, BM = 128;
constexpr int KBT = BM * 64;                        // a 128-row x 32-column bf16 tile: 64-byte rows, 64-byte swizzle
constexpr int AX_BYTES = BM * 32;                   // the extra k-step of a unit: 128 rows x 16 bf16, no swizzle
constexpr int WROWS = 96;                           // rows of a per-head QKV weight tile: q_h, k_h, v_h
constexpr int WQ_TILE = WROWS * 64;
constexpr int WX_TILE = WROWS * 32;                 // the extra k-step of a head's weights
constexpr int KV_SLOT = 2 * KBT;                    // k, v tiles of one item
constexpr int NBUF = 4, BUF_COLS = 96;              // item buffers of tensor memory
constexpr int ID_BYTES = 32 * 64;                   // the identity tile
constexpr int NRING = 4;                            // units whose row offsets are kept (a unit's epilogue runs long after its gather)
constexpr int kLoaderThreads = 128;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TM_Y = NBUF * BUF_COLS;          // the projection's accumulator (C columns) after the item buffers
constexpr uint32_t ROW_INVALID = 0xFFFFFFFFu;       // no such row (a padding row of the tile, or a window past the end)
constexpr int WIN_MISSING = 0, WIN_GATHER = 1, WIN_BOX = 2;
constexpr int N_BARS = 26;

struct FusedArgs {
  int n_windows, n_pairs, T, ws, shift, H, W;
  int nWw, nWh, win_per_img;
  FastDiv fd_wpi, fd_nww;
  int na;                                           // depth of the row ring (2 or 3)
  uint32_t smem_bytes;
  float eps, scale;
  const __nv_bfloat16 *x, *ln_g, *ln_b, *b_qkv, *b_proj, *table;
  __nv_bfloat16* y;
  int* status;
  int use_box;                                      // windows off the seam move as TMA boxes (the tensor map over x is valid)
  int split;                                        // first atom of rowmap that indexes the token inside its window (-1: evaluate every row in full)
  DevMap rowmap;                                    // row n T + i of the windowed view -> element offset of the token in x (and y)
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int NH, int KC>
__global__ void __launch_bounds__(32 * (9 + 4 * NH), 1)
swin_attn_fused_kernel(const __grid_constant__ CUtensorMap tmWq, const __grid_constant__ CUtensorMap tmWp,
                       const __grid_constant__ CUtensorMap tmX, const __grid_constant__ FusedArgs g) {
  constexpr int C = NH * D, NCH = C / 8;             // channels, 16-byte chunks per row
  constexpr int kThreads = 32 * (9 + 4 * NH);
  constexpr int A_BYTES = NH * KBT;                  // a unit's raw rows: NH k-blocks of 32 columns
  constexpr int WP_TILE = C * 64;                    // Wp[:, 32 h : 32 h + 32]: C rows x 64 bytes
  constexpr int BR = KC == 56 ? 28 : 36;             // 32-bit words per bias row (16-byte reads of 8 consecutive rows hit distinct banks)
  extern __shared__ uint8_t smem_raw[];
  const uint32_t pad = (1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  const int T = g.T, ws = g.ws, na = g.na;
  uint8_t* sA = smem;                                              // [na][NH k-blocks][8 KB]
  uint8_t* sKV = sA + na * A_BYTES;                                // [NH groups][k, v][8 KB]
  uint8_t* sWq = sKV + NH * KV_SLOT;                               // [NH heads][NH k-blocks][96 rows x 64 B]
  uint8_t* sWp = sWq + NH * NH * WQ_TILE;                          // [NH heads][C rows x 64 B]
  uint8_t* sAx = sWp + NH * WP_TILE;                               // [na][128 rows x 32 B]
  uint8_t* sWx = sAx + na * AX_BYTES;                              // [NH heads][96 rows x 32 B]
  uint8_t* sId = sWx + NH * WX_TILE;                               // [32 rows x 64 B]: the 32 x 32 identity (the residual rides on the tensor core)
  uint32_t* bias_s = reinterpret_cast<uint32_t*>(sId + ID_BYTES);  // [NH][T][BR]: bf16 pairs
  float* bp_s = reinterpret_cast<float*>(bias_s + NH * T * BR);    // [C]
  float* rstd_s = bp_s + C;                                        // [na][128]
  uint32_t* rowoff_s = reinterpret_cast<uint32_t*>(rstd_s + na * BM);   // [NRING][128]: row offset in 16-byte units
  float* ln_s = reinterpret_cast<float*>(rowoff_s + NRING * BM);   // [2][C]: gamma, beta
  int* tyx_s = reinterpret_cast<int*>(ln_s + 2 * C);               // [64]: ty << 8 | tx
  uint32_t* kmask_s = reinterpret_cast<uint32_t*>(tyx_s + TP);     // [4]
  int4* tok_s = reinterpret_cast<int4*>(kmask_s + 4);              // [64]: the map's contribution of token t: (offset, u0, u1, -)
  int4* win_s = tok_s + TP;                                        // [2 units][2 windows]: the contribution of window n: (offset lo, hi, u0, u1)
  int* wkind_s = reinterpret_cast<int*>(win_s + 4);                // [na][2 windows] (+ pad): how the window's rows come in
  uint64_t* bars = reinterpret_cast<uint64_t*>(wkind_s + 8);
  uint64_t* w_full = bars;
  uint64_t *a_full = bars + 1, *a_free = a_full + 3, *landed = a_free + 3;     // [3] each: per slot of the row ring
  uint64_t *s_full = landed + 3, *o_full = s_full + 3;             // [3] each: per group (the group issues these products itself)
  uint64_t *acc_full = o_full + 3, *ob_full = acc_full + NBUF;     // [NBUF] each: per item buffer (items 4 apart share one)
  uint64_t *y_full = ob_full + NBUF, *y_empty = y_full + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(y_empty + 1);
  int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);
  uint16_t* raw_s = reinterpret_cast<uint16_t*>(sKV);              // prologue scratch: the raw table columns, [NH][256]

  if (pad + (uint32_t)(reinterpret_cast<uint8_t*>(tmem_slot + 4) - smem) > g.smem_bytes) {
    if (threadIdx.x == 0) atomicExch(g.status, (int)SMARTMEM_ERR_UNSUPPORTED);
    return;
  }

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0);   // (provably warp-uniform: the issuing code below keeps its operands in uniform registers)
  // A CTA takes a contiguous run of window pairs.  (Dealing the pairs out round-robin looks equivalent but is not: with 32 pairs
  // per image and a stride of 148 a CTA sees the same pairs of every image, so a quarter of the CTAs got nothing but seam
  // windows -- the slow path: gathered rows and masked scores -- and finished microseconds after the rest.)
  const int uq = g.n_pairs / (int)gridDim.x, urem = g.n_pairs - uq * (int)gridDim.x;
  const int U = uq + ((int)blockIdx.x < urem ? 1 : 0);                              // units of this CTA
  const int ubase = (int)blockIdx.x * uq + ((int)blockIdx.x < urem ? (int)blockIdx.x : urem);   // its first pair
  const int total = U * NH;                                                         // items
  const float LOG2E = 1.4426950408889634f;

  if (tid == 0) {
    ptx::mbar_init(w_full, 1);
#pragma unroll 1
    for (int i = 0; i < 3; ++i) {
      ptx::mbar_init(&a_full[i], 4);
      ptx::mbar_init(&a_free[i], NH + 1);
      ptx::mbar_init(&landed[i], 4);
      ptx::mbar_init(&s_full[i], 1);
      ptx::mbar_init(&o_full[i], 1);
    }
#pragma unroll 1
    for (int i = 0; i < NBUF; ++i) {
      ptx::mbar_init(&acc_full[i], 1);
      ptx::mbar_init(&ob_full[i], 4);
    }
    ptx::mbar_init(y_full, 1);
    ptx::mbar_init(y_empty, 4);
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    // the weights do not depend on the kernel before this one: fetch them right away
    ptx::prefetch_tensormap(&tmWq);
    ptx::prefetch_tensormap(&tmWp);
    ptx::prefetch_tensormap(&tmX);
    ptx::mbar_expect_tx(w_full, (uint32_t)(NH * NH * WQ_TILE + NH * WP_TILE));
#pragma unroll 1
    for (int h = 0; h < NH; ++h)                       // (head, k-block, q / k / v): a box of 32 weight rows x 32 columns
#pragma unroll 1
      for (int kb = 0; kb < NH; ++kb)
#pragma unroll
        for (int which = 0; which < 3; ++which)
          ptx::tma_load_2d(sWq + (h * NH + kb) * WQ_TILE + which * (D * 64), &tmWq, w_full, kb * D, which * C + h * D);
#pragma unroll 1
    for (int h = 0; h < NH; ++h) ptx::tma_load_2d(sWp + h * WP_TILE, &tmWp, w_full, h * D, 0);
  }
  if (warp == 0) ptx::tmem_alloc(tmem_slot, TMEM_COLS);
  // parameter-only tables
  const int n_table = (2 * ws - 1) * (2 * ws - 1);
  for (int i = tid; i < NH * 256; i += kThreads) {
    const int h = i >> 8, e = i & 255;
    raw_s[i] = e < n_table ? reinterpret_cast<const uint16_t*>(g.table)[e * NH + h] : (uint16_t)0;
  }
  if (tid < TP) {
    tyx_s[tid] = ((tid / ws) << 8) | (tid % ws);
    int4 tk = make_int4(0, 0, 0, 0);
    if (g.split >= 0 && tid < T) {
      const DevMapPart pt = devmap_part_rolled(g.rowmap, g.split, g.rowmap.n_atoms, (uint32_t)tid);
      tk = make_int4((int)pt.off, pt.u0, pt.u1, 0);
    }
    tok_s[tid] = tk;
  }
  for (int i = tid; i < C; i += kThreads) {
    ln_s[i] = __bfloat162float(g.ln_g[i]);
    ln_s[C + i] = __bfloat162float(g.ln_b[i]);
    bp_s[i] = __bfloat162float(g.b_proj[i]);
  }
  for (int i = tid; i < na * A_BYTES / 16; i += kThreads) reinterpret_cast<uint4*>(sA)[i] = make_uint4(0, 0, 0, 0);
  for (int i = tid; i < na * AX_BYTES / 16; i += kThreads) reinterpret_cast<uint4*>(sAx)[i] = make_uint4(0, 0, 0, 0);
  for (int i = tid; i < ID_BYTES / 16; i += kThreads) reinterpret_cast<uint4*>(sId)[i] = make_uint4(0, 0, 0, 0);
  for (int i = tid; i < na * BM; i += kThreads) rstd_s[i] = 0.f;
  for (int i = tid; i < NRING * BM; i += kThreads) rowoff_s[i] = ROW_INVALID;
  __syncthreads();
  if (tid < 32)                                       // identity: row n has a one in column n
    *reinterpret_cast<uint16_t*>(sId + sw64_off(tid, tid >> 3) + (tid & 7) * 2) = 0x3F80u;
  // keys below / right of the wrap line of a seam window (bit c = key c)
  if (warp == 2) {
    const int c0 = lane, c1 = lane + 32;
    const bool y0 = c0 < T && (tyx_s[c0] >> 8) >= ws - g.shift, y1 = c1 < T && (tyx_s[c1] >> 8) >= ws - g.shift;
    const bool x0 = c0 < T && (tyx_s[c0] & 255) >= ws - g.shift, x1 = c1 < T && (tyx_s[c1] & 255) >= ws - g.shift;
    const uint32_t m0 = __ballot_sync(0xFFFFFFFFu, y0), m1 = __ballot_sync(0xFFFFFFFFu, y1);
    const uint32_t m2 = __ballot_sync(0xFFFFFFFFu, x0), m3 = __ballot_sync(0xFFFFFFFFu, x1);
    if (lane == 0) { kmask_s[0] = m0; kmask_s[1] = m1; kmask_s[2] = m2; kmask_s[3] = m3; }
  }
  // fold gamma into the resident QKV weights; the column terms c_n and b'_n go into the extra k-step (thread = one weight row)
  const bool w_ok = ptx::mbar_wait(w_full, 0, abort_flag, g.status);
  if (w_ok && tid < 2 * NH * WROWS) {                  // (whole warps: 2 * NH * 96 is a multiple of 32)
    const int row = tid >> 1, half = tid & 1;          // two threads per weight row: the first and second half of its chunks
    const int h = row / WROWS, rr = row - h * WROWS;
    const int which = rr >> 5, j = rr & 31;
    float csum = 0.f, bsum = half ? 0.f : __bfloat162float(g.b_qkv[which * C + h * D + j]);
    float bsum2 = 0.f;
#pragma unroll 2
    for (int ci = half * (NCH / 2); ci < (half + 1) * (NCH / 2); ++ci) {     // chunk ci of the row: k-block ci / 4, chunk ci % 4
      uint4* p = reinterpret_cast<uint4*>(sWq + (h * NH + (ci >> 2)) * WQ_TILE + sw64_off(rr, ci & 3));
      const uint4 wv = *p;
      const uint32_t w4[4] = {wv.x, wv.y, wv.z, wv.w};
      const float4 ga0 = *reinterpret_cast<const float4*>(ln_s + ci * 8), ga1 = *reinterpret_cast<const float4*>(ln_s + ci * 8 + 4);
      const float4 be0 = *reinterpret_cast<const float4*>(ln_s + C + ci * 8), be1 = *reinterpret_cast<const float4*>(ln_s + C + ci * 8 + 4);
      const float ga[8] = {ga0.x, ga0.y, ga0.z, ga0.w, ga1.x, ga1.y, ga1.z, ga1.w};
      const float be[8] = {be0.x, be0.y, be0.z, be0.w, be1.x, be1.y, be1.z, be1.w};
      uint32_t o4[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 f = bf16x2_to_float2(w4[e]);
        bsum = fmaf(be[2 * e], f.x, bsum);
        bsum2 = fmaf(be[2 * e + 1], f.y, bsum2);
        o4[e] = float2_to_bf16x2(ga[2 * e] * f.x, ga[2 * e + 1] * f.y);
        const float2 r2 = bf16x2_to_float2(o4[e]);
        csum += r2.x + r2.y;
      }
      *p = make_uint4(o4[0], o4[1], o4[2], o4[3]);
    }
    bsum += bsum2;
    csum += __shfl_xor_sync(0xFFFFFFFFu, csum, 1);
    bsum += __shfl_xor_sync(0xFFFFFFFFu, bsum, 1);
    if (half == 0) {
      uint4 k0, k1;
      extra_col(csum, bsum, k0, k1);
      *reinterpret_cast<uint4*>(sWx + h * WX_TILE + plain_off(rr, 0)) = k0;
      *reinterpret_cast<uint4*>(sWx + h * WX_TILE + plain_off(rr, 1)) = k1;
    }
  }
  if (tid < 2 && U > 0 && g.split >= 0) {              // the first unit's windows under the map (parameters only)
    const int n = 2 * ubase + tid;
    int4 wp = make_int4(0, 0, 0, 0);
    if (n < g.n_windows) {
      const DevMapPart pw = devmap_part_rolled(g.rowmap, 0, g.split, (uint32_t)n);
      wp = make_int4((int)(uint32_t)(pw.off & 0xFFFFFFFFll), (int)(pw.off >> 32), pw.u0, pw.u1);
    }
    win_s[tid] = wp;
  }
  ptx::fence_proxy_async();                           // the rewritten weights -> visible to the MMAs
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                                         // everything above depends on parameters only
  pdl_launch_dependents();

  if (warp < 4) {
    // ---- rows of the units ahead -> the operand layout in shared memory ------------------------------------------------------
    const int lt = tid;                                // 0 .. 127
    constexpr int RPI = kLoaderThreads / NCH;          // rows per round of the gather loop: a row by NCH consecutive threads
    const int my_ch = lt % NCH, my_slot = lt / NCH;
    bool ok = true;
    auto vote = [&](bool pred, bool all) {             // OR (all = false) or AND (all = true) over the loader threads; also a barrier
      uint32_t res;
      if (all)
        asm volatile("{\n\t.reg .pred pin, pout;\n\tsetp.ne.u32 pin, %1, 0;\n\tbar.red.and.pred pout, 1, 128, pin;\n\tselp.u32 %0, 1, 0, pout;\n\t}"
                     : "=r"(res) : "r"(pred ? 1u : 0u) : "memory");
      else
        asm volatile("{\n\t.reg .pred pin, pout;\n\tsetp.ne.u32 pin, %1, 0;\n\tbar.red.or.pred pout, 1, 128, pin;\n\tselp.u32 %0, 1, 0, pout;\n\t}"
                     : "=r"(res) : "r"(pred ? 1u : 0u) : "memory");
      return res != 0;
    };
    auto window_part = [&](int ul) {                   // threads 0, 1: the leading atoms' contribution of the unit's two windows
      if (lt < 2 && ul < U && g.split >= 0) {
        const int n = 2 * (ubase + ul) + lt;
        int4 wp = make_int4(0, 0, 0, 0);
        if (n < g.n_windows) {
          const DevMapPart pw = devmap_part_rolled(g.rowmap, 0, g.split, (uint32_t)n);
          wp = make_int4((int)(uint32_t)(pw.off & 0xFFFFFFFFll), (int)(pw.off >> 32), pw.u0, pw.u1);
        }
        win_s[(ul & 1) * 2 + lt] = wp;
      }
    };
    auto issue_loads = [&](int ul) {
      const int ab = ul % na;
      const int p = ubase + ul;
      {                                                 // a thread per row of the pair tile: the window's kind, the row's offset
        const int w = lt >> 6, i = lt & 63, n = 2 * p + w;
        int kind = WIN_MISSING, wy = 0, wx = 0, b = 0;
        if (n < g.n_windows) {
          b = (int)fd_div((uint32_t)n, g.fd_wpi);
          const int wl = n - b * g.win_per_img;
          wy = (int)fd_div((uint32_t)wl, g.fd_nww);
          wx = wl - wy * g.nWw;
          const bool seam = g.shift > 0 && (wy == g.nWh - 1 || wx == g.nWw - 1);
          kind = (seam || !g.use_box) ? WIN_GATHER : WIN_BOX;
        }
        uint32_t off16 = ROW_INVALID;
        if (i < T && kind != WIN_MISSING) {            // the offset under the map: the gather of a seam window, the residual and the scatter use it
          long long off;
          if (g.split >= 0) {
            const int4 wp = win_s[(ul & 1) * 2 + w], tk = tok_s[i];
            const long long woff = (long long)(((unsigned long long)(uint32_t)wp.y << 32) | (uint32_t)wp.x);
            off = devmap_finish2(g.rowmap, woff + tk.x, wp.z + tk.y, wp.w + tk.z);
          } else {
            off = devmap_eval_unrolled(g.rowmap, (uint32_t)(n * T + i));
          }
          off16 = (uint32_t)(off >> 3);
        }
        rowoff_s[(ul % NRING) * BM + lt] = off16;
        if (i == 0) {
          wkind_s[ab * 2 + w] = kind;
          if (kind == WIN_BOX) {                        // this thread moves the window (no arrival: the loader warps arrive below)
            ptx::mbar_add_tx(&landed[ab], (uint32_t)(T * C * 2));
#pragma unroll
            for (int kb = 0; kb < NH; ++kb)
              ptx::tma_load_4d(sA + ab * A_BYTES + kb * KBT + w * (64 * 64), &tmX, &landed[ab], kb * D, wx * ws + g.shift,
                               wy * ws + g.shift, b);
          }
        }
      }
      asm volatile("bar.sync 2, 128;" ::: "memory");
      const int kind0 = wkind_s[ab * 2], kind1 = wkind_s[ab * 2 + 1];
      if (kind0 != WIN_BOX || kind1 != WIN_BOX) {
        uint8_t* tile = sA + ab * A_BYTES + (my_ch >> 2) * KBT;
        for (int v = my_slot; v < 2 * T && my_slot < RPI; v += RPI) {
          const int w = v >= T ? 1 : 0, row = w * 64 + (v - w * T);
          const int kind = w ? kind1 : kind0;
          uint8_t* dst = tile + sw64_off(row, my_ch & 3);
          if (kind == WIN_MISSING) *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);    // no stale rows
          else if (kind == WIN_GATHER)
            ptx::cp_async16(dst, g.x + ((size_t)rowoff_s[(ul % NRING) * BM + row] << 3) + my_ch * 8);
        }
      }
      ptx::cp_async_commit();
      window_part(ul + 1);                             // read after the next barrier of the loader threads
    };
    auto statistics = [&](int ul) {
      const int ab = ul % na;
      const int r = lt, i = lt & 63;
      if (i < T) {
        float rstd = 0.f;
        uint4 k0 = make_uint4(0, 0, 0, 0), k1 = k0;
        if (rowoff_s[(ul % NRING) * BM + r] != ROW_INVALID) {
          // two passes over the row in shared memory (mean, then squared deviations); the loops are only partly unrolled: this code
          // runs once per unit, and fetching its instructions costs as much as executing them
          f32x2 s2[2] = {0ull, 0ull};
#pragma unroll 4
          for (int ch = 0; ch < NCH; ++ch) {
            const uint4 xv = *reinterpret_cast<const uint4*>(sA + ab * A_BYTES + (ch >> 2) * KBT + sw64_off(r, ch & 3));
            const uint32_t x4[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
              s2[e & 1] = ptx::add2(s2[e & 1], ptx::pack2(__uint_as_float(x4[e] << 16), __uint_as_float(x4[e] & 0xFFFF0000u)));
          }
          float a0, a1, a2, a3;
          ptx::unpack2(s2[0], a0, a1);
          ptx::unpack2(s2[1], a2, a3);
          const float mean = ((a0 + a1) + (a2 + a3)) * (1.0f / (float)C);
          const f32x2 nm2 = ptx::pack2(-mean, -mean);
          f32x2 q2[2] = {0ull, 0ull};
#pragma unroll 4
          for (int ch = 0; ch < NCH; ++ch) {
            const uint4 xv = *reinterpret_cast<const uint4*>(sA + ab * A_BYTES + (ch >> 2) * KBT + sw64_off(r, ch & 3));
            const uint32_t x4[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const f32x2 d2 = ptx::add2(ptx::pack2(__uint_as_float(x4[e] << 16), __uint_as_float(x4[e] & 0xFFFF0000u)), nm2);
              q2[e & 1] = ptx::fma2(d2, d2, q2[e & 1]);
            }
          }
          ptx::unpack2(q2[0], a0, a1);
          ptx::unpack2(q2[1], a2, a3);
          const float var = ((a0 + a1) + (a2 + a3)) * (1.0f / (float)C) + g.eps;
          rstd = rsqrtf(var);
          extra_row(-mean, var * rstd, k0, k1);          // sigma = var / sqrt(var)
        }
        rstd_s[ab * BM + r] = rstd;
        *reinterpret_cast<uint4*>(sAx + ab * AX_BYTES + plain_off(r, 0)) = k0;
        *reinterpret_cast<uint4*>(sAx + ab * AX_BYTES + plain_off(r, 1)) = k1;
      }
      ptx::fence_proxy_async();                        // the extra k-step -> visible to the MMAs
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&a_full[ab]);
    };
    // A unit's rows are requested as soon as its ring slot is free (the QKV products of the unit that held it are done); when
    // no slot is free the oldest request in flight is waited for and handed to the statistics warps.
    int issued = 0, done = 0;
    while (done < U) {
      if (issued < U && issued - done < na) {
        uint64_t* bar = &a_free[issued % na];
        const uint32_t par = (uint32_t)(((issued / na) & 1) ^ 1);
        bool ready;
        if (issued == done) {
          ok = ptx::mbar_wait_relaxed(bar, par, abort_flag, g.status, 64);
          if (vote(!ok, false)) break;
          ready = true;
        } else {
          ready = vote(ptx::mbar_test(bar, par), true);
        }
        if (ready) {
          issue_loads(issued);
          ++issued;
          continue;
        }
      }
      const int pending = issued - done;               // cp.async groups in flight; the oldest belongs to unit `done`
      if (pending >= 3) ptx::cp_async_wait<2>();
      else if (pending == 2) ptx::cp_async_wait<1>();
      else ptx::cp_async_wait<0>();
      ptx::fence_proxy_async();                        // the gathered rows -> visible to the MMAs
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&landed[done % na]);
      // every row of the unit is in (the loader warps' copies and the TMA boxes): its statistics, a thread per row
      ok = ptx::mbar_wait_relaxed(&landed[done % na], (done / na) & 1, abort_flag, g.status, 32);
      if (vote(!ok, false)) break;
      statistics(done);
      ++done;
    }
  } else if (warp < 4 + 4 * NH) {
    // ---- row groups: group h takes head h of every unit; one row of the pair tile per thread.  The group's elected thread issues
    // the item's S, P V and projection products, and the QKV product of its NEXT item as soon as the tensor-memory buffer that
    // item rotates into is free (the projection of the item before this one has completed). ------------------------------------
    const int gi = (warp - 4) >> 2;                    // group = head
    const int q = warp & 3;                            // TMEM lane quadrant
    const int r = q * 32 + lane;
    const int w = r >> 6, i = r & 63;                  // window of the pair, token
    const bool elected = q == 0 && lane == 0;          // (arrivals on behalf of the group)
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    const int my_ty = tyx_s[i] >> 8, my_tx = tyx_s[i] & 255;
    const uint32_t ky_lo = kmask_s[0], ky_hi = kmask_s[1], kx_lo = kmask_s[2], kx_hi = kmask_s[3];
    const uint32_t my_fy = my_ty >= ws - g.shift ? 0xFFFFFFFFu : 0u, my_fx = my_tx >= ws - g.shift ? 0xFFFFFFFFu : 0u;
    uint8_t* slot_base = sKV + gi * KV_SLOT;
    const uint32_t* brow = bias_s + (gi * T + (i < T ? i : 0)) * BR;
    const f32x2 scale2 = ptx::pack2(g.scale, g.scale), log2e2 = ptx::pack2(LOG2E, LOG2E);
    // This head's bias as a [T, T] table of bf16 pairs, -inf for the padded keys, built by the group itself while the first unit's
    // rows are on their way (a task = a quarter of a row).  The first group barrier below orders it before the first softmax.
    for (int task = (warp - 4 - 4 * gi) * 32 + lane; task < T * 4; task += 128) {
      const int r = task >> 2, qtr = task & 3;                        // row, quarter of the row's key pairs
      const int ry = tyx_s[r] >> 8, rx = tyx_s[r] & 255;
      const uint16_t* tab = raw_s + gi * 256 + (ry + ws - 1) * (2 * ws - 1) + (rx + ws - 1);
#pragma unroll 1
      for (int c2 = qtr * (KC / 8); c2 < (qtr + 1) * (KC / 8); ++c2) {
        uint32_t word = 0;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const int c = 2 * c2 + k;
          uint32_t bits = 0xFF80u;                       // -inf: padded keys never contribute
          if (c < T) {
            const int cyx = tyx_s[c];
            bits = tab[-(cyx >> 8) * (2 * ws - 1) - (cyx & 255)];
          }
          word |= bits << (16 * k);
        }
        bias_s[(gi * T + r) * BR + c2] = word;
      }
    }
    bool ok = true;
    auto group_sync = [&]() {                          // barrier of the group's 128 threads; true if one of them gave up waiting
      uint32_t gave_up;
      asm volatile(
          "{\n\t.reg .pred pin, pout;\n\t"
          "setp.ne.u32 pin, %2, 0;\n\t"
          "bar.red.or.pred pout, %1, 128, pin;\n\t"
          "selp.u32 %0, 1, 0, pout;\n\t}"
          : "=r"(gave_up)
          : "r"(3 + gi), "r"(ok ? 0u : 1u)
          : "memory");
      return gave_up != 0;
    };
    for (int ul = 0; ul < U; ++ul) {
      const int it = ul * NH + gi;
      const int ab = ul % na;
      const uint32_t tb = tmem_base + (it & (NBUF - 1)) * BUF_COLS + lane_addr;
      // -- q, k, v of this row: rstd times the accumulator (the mean and bias terms rode on the extra k-step) --
      ok = ok && GWAIT(&a_full[ab], (ul / na) & 1) &&     // (long complete: orders the read of rstd)
           GWAIT(&acc_full[it & (NBUF - 1)], (it >> 2) & 1);
      if (ok) {
        if (elected) ptx::mbar_arrive(&a_free[ab]);      // this head's product has read the unit's rows
        ptx::tc_fence_after();
        const float rstd = rstd_s[ab * BM + r];
        const f32x2 r2 = ptx::pack2(rstd, rstd);
        uint32_t rv[32], q16[16];
        auto scaled_pairs = [&](uint32_t* out) {         // 32 accumulator columns in rv -> 16 bf16 pairs of rstd * acc
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            float v0, v1;
            ptx::unpack2(ptx::mul2(ptx::pack2(__uint_as_float(rv[2 * c]), __uint_as_float(rv[2 * c + 1])), r2), v0, v1);
            out[c] = float2_to_bf16x2(v0, v1);
          }
        };
        ptx::tmem_ld32(tb, rv);                          // q
        ptx::tmem_ld_wait();
        scaled_pairs(q16);
#pragma unroll
        for (int kv = 0; kv < 2; ++kv) {                 // k, v -> this group's operand tiles
          uint32_t o16[16];
          ptx::tmem_ld32(tb + 32 + kv * 32, rv);
          ptx::tmem_ld_wait();
          scaled_pairs(o16);
#pragma unroll
          for (int c = 0; c < 4; ++c)
            *reinterpret_cast<uint4*>(slot_base + kv * KBT + sw64_off(r, c)) =
                make_uint4(o16[c * 4], o16[c * 4 + 1], o16[c * 4 + 2], o16[c * 4 + 3]);
        }
        // q as the S product's A operand: 64 bf16 = 32 packed columns over the accumulator's last 32 (v has been read): this
        // window's half carries q, the other half zeros (the two windows' keys are stacked along the reduction dimension)
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          rv[c] = w ? 0u : q16[c];
          rv[16 + c] = w ? q16[c] : 0u;
        }
        ptx::tmem_st32(tb + 64, rv);
        ptx::tmem_st_wait();
        ptx::fence_proxy_async();                      // generic-proxy writes -> visible to the MMAs
        ptx::tc_fence_before();
      }
      if (__any_sync(0xFFFFFFFFu, group_sync())) break;
      if (q == 0 && ptx::elect_one()) {
        // S = [q0 0; 0 q1] [k0 | k1]^T: four k16 steps, the first two over window 0's keys, the last two over window 1's
        ptx::tc_fence_after();
        const uint32_t idesc = ptx::make_idesc_bf16(BM, 64, false, false);
        const uint32_t d = tb - lane_addr, qa = d + 64;
        const uint64_t kd0 = desc_sw64(ptx::smem_u32(slot_base)), kd1 = desc_sw64(ptx::smem_u32(slot_base) + 64 * 64);
        ptx::tc_mma_bf16_ta(d, qa, kd0, idesc, 0u);
        ptx::tc_mma_bf16_ta(d, qa + 8, kd0 + 2, idesc, 1u);
        ptx::tc_mma_bf16_ta(d, qa + 16, kd1, idesc, 1u);
        ptx::tc_mma_bf16_ta(d, qa + 24, kd1 + 2, idesc, 1u);
        ptx::tc_commit(&s_full[gi]);
      }
      // -- seam mask of this row's window (shifted blocks: windows in the last window row or column) --
      const int n = 2 * (ubase + ul) + w;
      bool masked = false;
      uint32_t diff_lo = 0, diff_hi = 0;
      if (g.shift > 0 && n < g.n_windows) {
        const int wl = n - (int)fd_div((uint32_t)n, g.fd_wpi) * g.win_per_img;
        const int wy = (int)fd_div((uint32_t)wl, g.fd_nww), wx = wl - wy * g.nWw;
        const bool last_row = wy == g.nWh - 1, last_col = wx == g.nWw - 1;
        masked = last_row || last_col;
        if (last_row) { diff_lo |= ky_lo ^ my_fy; diff_hi |= ky_hi ^ my_fy; }
        if (last_col) { diff_lo |= kx_lo ^ my_fx; diff_hi |= kx_hi ^ my_fx; }
      }
      // -- softmax of this row over its window's keys --
      ok = GWAIT(&s_full[gi], ul & 1);
      float inv = 0.f;
      if (ok) {
        ptx::tc_fence_after();
        uint32_t rv[KC];
        ptx::tmem_ld32(tb, rv);
        if constexpr (KC == 64) {
          ptx::tmem_ld32(tb + 32, rv + 32);
        } else {
          ptx::tmem_ld16(tb + 32, rv + 32);
          ptx::tmem_ld8(tb + 48, rv + 48);
        }
        ptx::tmem_ld_wait();
        float sc[KC];
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int v8 = 0; v8 < KC / 8; ++v8) {
          const uint4 b4 = *reinterpret_cast<const uint4*>(brow + v8 * 4);
          const uint32_t bw[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int c = v8 * 8 + 2 * j;
            ptx::unpack2(ptx::fma2(ptx::pack2(__uint_as_float(rv[c]), __uint_as_float(rv[c + 1])), scale2,
                                   ptx::pack2(__uint_as_float(bw[j] << 16), __uint_as_float(bw[j] & 0xFFFF0000u))),
                         sc[c], sc[c + 1]);
          }
        }
        if (masked) {                                  // keys of another region get -100
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            if ((diff_lo >> c) & 1u) sc[c] -= 100.f;
            if (c + 32 < KC && ((diff_hi >> c) & 1u)) sc[c + 32] -= 100.f;
          }
        }
#pragma unroll
        for (int c = 0; c < KC; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], sc[c]);
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        const float nmx = -mx * LOG2E;
        const f32x2 nmx2 = ptx::pack2(nmx, nmx);
        f32x2 sum2[2] = {0ull, 0ull};
        uint32_t pk[32];
#pragma unroll
        for (int c = KC / 2; c < 32; ++c) pk[c] = 0u;        // padding keys
#pragma unroll
        for (int c = 0; c < KC; c += 2) {
          float e0, e1;
          ptx::unpack2(ptx::fma2(ptx::pack2(sc[c], sc[c + 1]), log2e2, nmx2), e0, e1);
          const float p0 = ex2f(e0), p1 = ex2f(e1);
          sum2[(c >> 1) & 1] = ptx::add2(sum2[(c >> 1) & 1], ptx::pack2(p0, p1));
          pk[c / 2] = float2_to_bf16x2(p0, p1);
        }
        float s0, s1, s2, s3;
        ptx::unpack2(sum2[0], s0, s1);
        ptx::unpack2(sum2[1], s2, s3);
        inv = 1.f / ((s0 + s1) + (s2 + s3));
        // P row (bf16 pairs) over the score columns: this window's keys at packed columns 32 w .. 32 w + 31, zeros for the
        // other window's keys (block-diagonal P against the stacked values)
        ptx::tmem_st32(tb + w * 32, pk);
#pragma unroll
        for (int c = 0; c < 32; ++c) pk[c] = 0u;
        ptx::tmem_st32(tb + (1 - w) * 32, pk);
        ptx::tmem_st_wait();
        ptx::tc_fence_before();
      }
      if (__any_sync(0xFFFFFFFFu, group_sync())) break;
      if (q == 0 && ptx::elect_one()) {
        // O = P [v0; v1] over the columns q has left: P from tensor memory, V as it lies (MN-major B operand); 16 keys per
        // step: P +8 packed columns, V +16 rows = 1024 bytes
        ptx::tc_fence_after();
        const uint32_t idesc = ptx::make_idesc_bf16(BM, D, false, true);
        const uint64_t vd = desc_sw64(ptx::smem_u32(slot_base) + KBT);
        const uint32_t pa = tb - lane_addr, od = pa + 64;
        ptx::tc_mma_bf16_ta(od, pa, vd, idesc, 0u);
#pragma unroll
        for (int ks = 1; ks < 8; ++ks) ptx::tc_mma_bf16_ta(od, pa + 8 * ks, vd + ks * (1024 >> 4), idesc, 1u);
        ptx::tc_commit(&o_full[gi]);
      }
      // -- O row: normalise, bf16 pairs, back into tensor memory as the projection's A operand --
      ok = GWAIT(&o_full[gi], ul & 1);
      if (ok) {
        ptx::tc_fence_after();
        uint32_t rv[32], ob[16];
        const f32x2 inv2 = ptx::pack2(inv, inv);
        ptx::tmem_ld32(tb + 64, rv);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          float v0, v1;
          ptx::unpack2(ptx::mul2(ptx::pack2(__uint_as_float(rv[2 * e]), __uint_as_float(rv[2 * e + 1])), inv2), v0, v1);
          ob[e] = float2_to_bf16x2(v0, v1);
        }
        ptx::tmem_st16(tb + 64, ob);
        ptx::tmem_st_wait();
        ptx::tc_fence_before();
      }
      __syncwarp();
      if (!ok) break;
      if (lane == 0) ptx::mbar_arrive(&ob_full[it & (NBUF - 1)]);       // the projection of this item may be issued
    }
  } else if (warp == 8 + 4 * NH) {
    // ---- the products that have slack -- QKV of the items ahead, the projections -- are issued by a thread of their own, in item
    // order, so that no group thread ever waits on their inputs.  Issue order is accumulation order (the heads of a unit add
    // up in Y) and also orders a buffer's next accumulator behind the projection that reads the buffer last. -----------------
    if (__all_sync(0xFFFFFFFFu, w_ok ? 1 : 0)) {          // the whole warp walks the queues; an elected lane issues
      const uint32_t idesc_qkv = ptx::make_idesc_bf16(BM, WROWS, false, false);
      const uint32_t idesc_pj = ptx::make_idesc_bf16(BM, C, false, false);
      const uint32_t idesc_id = ptx::make_idesc_bf16(BM, D, false, false);
      const uint32_t a_base = ptx::smem_u32(sA), ax_base = ptx::smem_u32(sAx), wq_base = ptx::smem_u32(sWq);
      const uint32_t wx_base = ptx::smem_u32(sWx), wp_base = ptx::smem_u32(sWp);
      int qi = 0, qh = 0, qu = 0, qab = 0, qaph = 0;   // QKV queue: item, head, unit, row-ring slot and its phase
      int ji = 0, jh = 0, ju = 0;                      // projection queue
      int xu = 0, xab = 0, xaph = 0;                   // residual queue: unit, its row-ring slot and phase
      const uint32_t id_base = ptx::smem_u32(sId);
      uint32_t idle = 0;
      unsigned long long t_idle = 0;
      while (ji < total) {
        bool progress = false;
        if (xu < U && xu <= ju && __all_sync(0xFFFFFFFFu, ptx::mbar_test(y_empty, (xu & 1) ^ 1) && ptx::mbar_test(&a_full[xab], xaph))) {
          // Y = X I: the unit's raw rows open the accumulation (the epilogue of the unit before has read Y); exact, since every
          // product is a bf16 value times one.  The product is the last reader of the unit's rows: its completion frees the slot.
          ptx::tc_fence_after();
          const uint64_t bd = desc_sw64(id_base);
          const uint64_t ad0 = desc_sw64(a_base + xab * A_BYTES);
          if (ptx::elect_one()) {
#pragma unroll
            for (int kb = 0; kb < NH; ++kb) {          // 32 channels at a time: Y[:, 32 kb : 32 kb + 32] = X[:, 32 kb : 32 kb + 32] I_32
              const uint64_t ad = ad0 + kb * (KBT >> 4);
              ptx::tc_mma_bf16(tmem_base + TM_Y + kb * D, ad, bd, idesc_id, 0u);
              ptx::tc_mma_bf16(tmem_base + TM_Y + kb * D, ad + 2, bd + 2, idesc_id, 1u);
            }
            ptx::tc_commit(&a_free[xab]);
          }
          __syncwarp();
          ++xu;
          if (++xab == na) { xab = 0; xaph ^= 1; }
          progress = true;
        }
        if (xu > ju && __all_sync(0xFFFFFFFFu, ptx::mbar_test(&ob_full[ji & (NBUF - 1)], (ji >> 2) & 1))) {
          // Y += Ob_h Wp[:, 32 h : 32 h + 32]^T; the last head hands Y to the epilogue
          ptx::tc_fence_after();
          const uint32_t a = tmem_base + (ji & (NBUF - 1)) * BUF_COLS + 64;
          const uint64_t bd = desc_sw64(wp_base + jh * WP_TILE);
          if (ptx::elect_one()) {
            ptx::tc_mma_bf16_ta(tmem_base + TM_Y, a, bd, idesc_pj, 1u);
            ptx::tc_mma_bf16_ta(tmem_base + TM_Y, a + 8, bd + 2, idesc_pj, 1u);
            if (jh == NH - 1) ptx::tc_commit(y_full);
          }
          __syncwarp();
          ++ji;
          if (++jh == NH) { jh = 0; ++ju; }
          progress = true;
        }
        if (qi < total && qi < ji + NBUF && __all_sync(0xFFFFFFFFu, ptx::mbar_test(&a_full[qab], qaph))) {
          // acc = [X | e] [Wq_h; Wk_h; Wv_h | f]^T into the buffer item qi - NBUF has left (its projection was issued above)
          ptx::tc_fence_after();
          const uint32_t d = tmem_base + (qi & (NBUF - 1)) * BUF_COLS;
          const uint64_t ad0 = desc_sw64(a_base + qab * A_BYTES), bd0 = desc_sw64(wq_base + qh * NH * WQ_TILE);
          const uint64_t axd = desc_plain(ax_base + qab * AX_BYTES), wxd = desc_plain(wx_base + qh * WX_TILE);
          if (ptx::elect_one()) {
#pragma unroll
            for (int kb = 0; kb < NH; ++kb) {
              const uint64_t ad = ad0 + kb * (KBT >> 4), bd = bd0 + kb * (WQ_TILE >> 4);
              ptx::tc_mma_bf16(d, ad, bd, idesc_qkv, kb ? 1u : 0u);
              ptx::tc_mma_bf16(d, ad + 2, bd + 2, idesc_qkv, 1u);    // next 16 channels: +32 bytes
            }
            ptx::tc_mma_bf16(d, axd, wxd, idesc_qkv, 1u);
            ptx::tc_commit(&acc_full[qi & (NBUF - 1)]);
          }
          __syncwarp();
          ++qi;
          if (++qh == NH) {
            qh = 0; ++qu;
            if (++qab == na) { qab = 0; qaph ^= 1; }
          }
          progress = true;
        }
        if (progress) {
          idle = 0;
        } else if ((++idle & 255u) == 0) {
          if (__any_sync(0xFFFFFFFFu, *(volatile int*)abort_flag)) break;
          const unsigned long long now = __shfl_sync(0xFFFFFFFFu, ptx::globaltimer(), 0);
          if (idle == 256u) t_idle = now;
          else if (now - t_idle > ptx::wait_limit_ns(g.status)) {
            if (lane == 0) {
              *abort_flag = 1;
              atomicExch(g.status, (int)SMARTMEM_ERR_TIMEOUT);
            }
            break;
          }
        }
      }
    }
  } else {
    // ---- Y epilogue: Y already holds x_row + sum_h Ob_h Wp_h^T (the residual rode on the tensor core as a product with the
    // identity); add the bias, round once, store the row at its offset under the map.  One row per thread. ------------------
    const int q = warp & 3;
    const int r = q * 32 + lane;
    const int i = r & 63;
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    const bool wide_store = (reinterpret_cast<uintptr_t>(g.y) & 31) == 0;
    bool ok = true;
    for (int ul = 0; ul < U && ok; ++ul) {
      ok = ptx::mbar_wait_relaxed(y_full, ul & 1, abort_flag, g.status, 32);
      if (!ok) break;
      ptx::tc_fence_after();
      const uint32_t my_off = rowoff_s[(ul % NRING) * BM + r];
      const bool valid = i < T && my_off != ROW_INVALID;
      uint4* yg = reinterpret_cast<uint4*>(g.y + ((size_t)(valid ? my_off : 0u) << 3));
#pragma unroll 1
      for (int k = 0; k < NH; ++k) {                   // 32 columns = 4 chunks of the row at a time
        uint32_t rv[32];
        ptx::tmem_ld32(tmem_base + TM_Y + lane_addr + k * 32, rv);
        ptx::tmem_ld_wait();
        if (k == NH - 1) {                             // Y is in registers: the next unit's products may overwrite it
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(y_empty);
        }
        if (valid) {
          uint4 o_prev = make_uint4(0, 0, 0, 0);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const float4 b0 = *reinterpret_cast<const float4*>(bp_s + k * 32 + c * 8);
            const float4 b1 = *reinterpret_cast<const float4*>(bp_s + k * 32 + c * 8 + 4);
            const f32x2 bb[4] = {ptx::pack2(b0.x, b0.y), ptx::pack2(b0.z, b0.w), ptx::pack2(b1.x, b1.y), ptx::pack2(b1.z, b1.w)};
            uint32_t o4[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int col = c * 8 + 2 * e;
              float v0, v1;
              ptx::unpack2(ptx::add2(ptx::pack2(__uint_as_float(rv[col]), __uint_as_float(rv[col + 1])), bb[e]), v0, v1);
              o4[e] = float2_to_bf16x2(v0, v1);
            }
            // whole 32-byte sectors per store when y is aligned for it (rows are 128 or 192 bytes apart)
            if (wide_store) {
              if (c & 1) ptx::st_global_v8(yg + k * 4 + c - 1, o_prev, make_uint4(o4[0], o4[1], o4[2], o4[3]));
              else o_prev = make_uint4(o4[0], o4[1], o4[2], o4[3]);
            } else {
              yg[k * 4 + c] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
            }
          }
        }
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace

// shared memory of a CTA with a row ring of `na` slots
static size_t fused_smem_need(int NH, int T, int na) {
  const int C = NH * D, br = T <= 56 ? 28 : 36;
  return (size_t)na * NH * KBT + (size_t)NH * KV_SLOT + (size_t)NH * NH * WQ_TILE + (size_t)NH * C * 64 +
         (size_t)na * AX_BYTES + (size_t)NH * WX_TILE + (size_t)ID_BYTES + (size_t)NH * T * br * 4 + (size_t)C * 4 +
         (size_t)na * BM * 4 + (size_t)NRING * BM * 4 + (size_t)2 * C * 4 + TP * 4 + 16 + TP * 16 + 4 * 16 + 32 + N_BARS * 8 + 16;
}
static constexpr size_t kMaxSmem = 232448;

bool swin_attn_fused_supported(int dtype, int C, int heads, int window) {
  return dtype == SMARTMEM_BF16 && (heads == 2 || heads == 3) && C == heads * D && window * window <= TP && window >= 1 &&
         fused_smem_need(heads, window * window, 2) <= kMaxSmem;
}

int launch_swin_attn_fused(const smartmem_swin_params_t& p, const DevMap& rowmap, const void* x, void* y, cudaStream_t st) {
  if (!swin_attn_fused_supported(p.dtype, p.C, p.heads, p.window)) return SMARTMEM_ERR_UNSUPPORTED;
  const int NH = p.heads, C = p.C, T = p.window * p.window;
  const long long n_windows = (long long)p.B * (p.H / p.window) * (p.W / p.window);
  if (n_windows < 1 || n_windows * T >= (1ll << 31) || (long long)p.B * p.H * p.W * C >= (1ll << 34)) return SMARTMEM_ERR_UNSUPPORTED;
  const void* ptrs[] = {x, y, p.ln1_g, p.ln1_b, p.w_qkv, p.b_qkv, p.w_proj, p.b_proj};
  for (const void* q : ptrs)
    if (!q || ((uintptr_t)q & 15)) return SMARTMEM_ERR_ALIGNMENT;
  if (!p.rel_bias_table) return SMARTMEM_ERR_INVALID_ARG;
  CUtensorMap twq, twp, tx;
  int rc;
  if ((rc = tc_encode_2d_sw64(p.w_qkv, C, 3 * C, C, D, D, &twq)) != SMARTMEM_OK) return rc;
  if ((rc = tc_encode_2d_sw64(p.w_proj, C, C, C, D, C, &twp)) != SMARTMEM_OK) return rc;
  memset(&tx, 0, sizeof(tx));
  const long long dims[4] = {C, p.W, p.H, p.B}, strides[3] = {C, (long long)p.W * C, (long long)p.H * p.W * C};
  const int box[4] = {D, p.window, p.window, 1};
  const bool use_box = tc_encode_nd_sw64(x, 4, dims, strides, box, &tx) == SMARTMEM_OK;
  FusedArgs g;
  memset(&g, 0, sizeof(g));
  g.use_box = use_box ? 1 : 0;
  g.n_windows = (int)n_windows;
  g.n_pairs = (int)((n_windows + 1) / 2);
  g.T = T; g.ws = p.window; g.shift = p.shift; g.H = p.H; g.W = p.W;
  g.nWw = p.W / p.window; g.nWh = p.H / p.window; g.win_per_img = g.nWw * g.nWh;
  g.fd_wpi = make_fastdiv((uint32_t)g.win_per_img);
  g.fd_nww = make_fastdiv((uint32_t)g.nWw);
  g.eps = p.ln_eps;
  g.scale = 1.0f / sqrtf((float)D);
  g.x = (const __nv_bfloat16*)x; g.y = (__nv_bfloat16*)y;
  g.ln_g = (const __nv_bfloat16*)p.ln1_g; g.ln_b = (const __nv_bfloat16*)p.ln1_b;
  g.b_qkv = (const __nv_bfloat16*)p.b_qkv; g.b_proj = (const __nv_bfloat16*)p.b_proj;
  g.table = (const __nv_bfloat16*)p.rel_bias_table;
  g.rowmap = rowmap;
  g.split = devmap_split(rowmap, T);
  g.status = device_status_ptr();
  if (!g.status) return SMARTMEM_ERR_CUDA;
  const bool kc56 = T <= 56;
  auto need = [&](int na) { return fused_smem_need(NH, T, na); };
  g.na = need(3) <= kMaxSmem ? 3 : 2;
  if (need(g.na) > kMaxSmem) return SMARTMEM_ERR_UNSUPPORTED;
  const size_t smem = need(g.na) + 1024 <= kMaxSmem ? need(g.na) + 1024 : kMaxSmem;   // alignment slack only while it fits
  g.smem_bytes = (uint32_t)smem;
  const void* fn = NH == 3 ? (kc56 ? (const void*)swin_attn_fused_kernel<3, 56> : (const void*)swin_attn_fused_kernel<3, 64>)
                           : (kc56 ? (const void*)swin_attn_fused_kernel<2, 56> : (const void*)swin_attn_fused_kernel<2, 64>);
  if ((rc = ensure_max_dynamic_smem(fn, (int)kMaxSmem)) != SMARTMEM_OK) return rc;
  const int sms = tc_sm_count();
  const unsigned grid = (unsigned)(g.n_pairs < sms ? g.n_pairs : sms);
  const unsigned threads = 32u * (9 + 4 * NH);
  profile_tick("attn_half_fused", st);
  cudaError_t e;
  if (NH == 3) e = kc56 ? launch_pdl(swin_attn_fused_kernel<3, 56>, dim3(grid), dim3(threads), smem, st, twq, twp, tx, g)
                        : launch_pdl(swin_attn_fused_kernel<3, 64>, dim3(grid), dim3(threads), smem, st, twq, twp, tx, g);
  else e = kc56 ? launch_pdl(swin_attn_fused_kernel<2, 56>, dim3(grid), dim3(threads), smem, st, twq, twp, tx, g)
                : launch_pdl(swin_attn_fused_kernel<2, 64>, dim3(grid), dim3(threads), smem, st, twq, twp, tx, g);
  count_launch();
  return e == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

}  // namespace smartmem
