// Fused MLP half of a transformer block on tcgen05:
//
//   out = residual + GELU(LN(A) W1^T + b1) W2^T + b2,     A [M, C], W1 [hidden, C], W2 [C, hidden]
//
// for narrow blocks (C in {64, 96}), where the hidden activation [M, hidden] is four times larger
// than everything else the block touches.  Neither the normalised rows nor the hidden tensor leave
// the SM.  Per 128-row tile: the producer brings the raw rows in by TMA, four warps normalise them
// in place (LayerNorm, a row per thread); then the kernel walks over chunks of 128 hidden columns:
// fc1 of a chunk accumulates in TMEM, the GELU warps add the bias, apply GELU on packed bf16 pairs
// and write the bf16 chunk back into the same TMEM buffer, and fc2 takes it from there as its A
// operand (tensor memory) while fc1 of the next chunk is already running.  The output accumulator is
// double-buffered in TMEM, so the output warps (bias, residual, row stores) overlap the next tile.
//
// Warp roles: 0 TMA producer (A tile double-buffered across tiles, weights streamed from L2 through
// a 4-stage ring in the order the two issuers consume them), 1 fc1 issuer + TMEM owner, 2-9 GELU
// (two warps per TMEM lane quadrant, 64 hidden columns each), 10-13 output, 14 fc2 issuer, 15-18
// LayerNorm.
//
// What bounds it (measured with clock stamps at every hand-off): the loop fc1(j) -> GELU(j) -> fc2(j) ->
// fc1(j+2) over the two S1/H buffers, about 2500 cycles per chunk.  The arithmetic in it is short
// (with the GELU arithmetic compiled out the chunk period stays near 2400 cycles and the kernel
// is only 15 % faster); most of it is the three hand-offs of the loop, each of which waits for the
// slowest of eight warps or for an issuer thread to be scheduled.  A variant with H in a buffer of
// its own (so that fc1(j+2) need not wait for fc2(j), but the H store waits for fc2(j-1)) ran at
// the same speed; a third S1 buffer does not fit the 512 columns next to the double-buffered
// output.  The floor under all of it is the special-function unit (tanh at 16 elements per clock
// per SM: about 1000 cycles per chunk).

#include "gemm_tc.cuh"
#include "ptx.cuh"


namespace smartmem {
namespace {

constexpr int BM = 128, BK = 64, HC = 128;         // tile rows, k-block, hidden chunk
constexpr int KB_BYTES = BM * BK * 2;              // one 128 x 64 bf16 operand block: 16 KB
constexpr int NST = 4;                             // weight ring stages; one stage = both k-blocks of a chunk's W1 or W2
constexpr int WST_BYTES = 2 * KB_BYTES;
constexpr int kGeluWarps = 8, kOutWarps = 4, kNormWarps = 4, kThreads = 32 * (3 + kGeluWarps + kOutWarps + kNormWarps);
constexpr uint32_t TM_S1 = 0, TM_OUT = 256, OUT_STRIDE = 96, TMEM_COLS = 512;   // S1 x2 (128; H is written over its own S1 buffer), OUT x2 (96)
constexpr int SMEM_TILES = (4 + 2 * NST) * KB_BYTES;         // A (2 buffers), weight ring
constexpr int N_BARS = 4 + 2 * NST + 2 + 2 + 2 + 4 + 2;

struct MlpArgs {
  int M, C, hidden, n_chunks, tiles;
  uint32_t smem_bytes;
  const __nv_bfloat16 *b1, *b2, *residual;
  const __nv_bfloat16 *ln_gamma, *ln_beta;         // LayerNorm applied to the rows of A on their way in (null: A is used as is)
  float ln_eps;
  __nv_bfloat16* out;
  int* status;
};

// tanh-form GELU (times two, see below) of two pre-activations, evaluated on packed bf16 pairs: the result is stored as
// bf16 anyway, and the packed path costs one conversion, four packed multiply-adds and one
// tanh.approx per PAIR, where the fp32 form costs seven instructions per element.  These warps are
// what bounds the kernel, and they are bound by instruction issue and by the special-function unit.
__device__ __forceinline__ uint32_t gelu_tanh_bf16x2(float a, float b) {
  const uint32_t u = float2_to_bf16x2(a, b);
  constexpr uint32_t C0 = 0x3F4C3F4Cu, C1 = 0x3D123D12u;   // 0.7979, 0.03568
  uint32_t u2, p, in, t, r;
  asm("mul.rn.bf16x2 %0, %1, %1;" : "=r"(u2) : "r"(u));
  asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(p) : "r"(C1), "r"(u2), "r"(C0));
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(in) : "r"(u), "r"(p));
  asm("tanh.approx.bf16x2 %0, %1;" : "=r"(t) : "r"(in));
  // u (1 + tanh) = TWICE the GELU: the factor 1/2 is a power of two, so it commutes with every rounding on the way and is
  // applied for free where the output warps add b2 (one multiply-add instead of one add); a multiply per pair saved here
  asm("fma.rn.bf16x2 %0, %1, %2, %1;" : "=r"(r) : "r"(u), "r"(t));
  return r;
}

// n <= 4 k16 steps of one 64-wide k-block; both operands K-major with the 128-byte swizzle, so a
// k16 step moves the descriptors' start address by 32 bytes (2 in descriptor units).
__device__ __forceinline__ void issue_kblock(uint32_t d_tmem, uint64_t ad0, uint64_t bd0, uint32_t idesc, int n, bool acc_first) {
  ptx::tc_mma_bf16(d_tmem, ad0, bd0, idesc, acc_first ? 1u : 0u);
#pragma unroll
  for (int k = 1; k < BK / 16; ++k)
    if (k < n) ptx::tc_mma_bf16(d_tmem, ad0 + 2 * k, bd0 + 2 * k, idesc, 1u);
}

__global__ void __launch_bounds__(kThreads, 1)
mlp_fused_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW1,
                 const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ MlpArgs g) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t pad = (1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  uint8_t* sA = smem;                              // [2 bufs][2 k-blocks][16 KB]
  uint8_t* sW = sA + 4 * KB_BYTES;                 // [NST][2 k-blocks][16 KB]
  uint64_t* bars = reinterpret_cast<uint64_t*>(sW + NST * WST_BYTES);
  uint64_t *a_full = bars, *a_empty = bars + 2, *w_full = bars + 4, *w_empty = w_full + NST;
  uint64_t *s1_full = w_empty + NST, *s1_empty = s1_full + 2, *h_full = s1_empty + 2;
  uint64_t *out_full = h_full + 2, *out_empty = out_full + 2, *a_ready = out_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(a_ready + 2);
  int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);
  float* b1_s = reinterpret_cast<float*>(tmem_slot + 4);     // [hidden]
  float* b2_s = b1_s + g.hidden;                             // [C]
  float* ln_s = b2_s + g.C;                                  // [2][C]: gamma, beta
  const bool fuse_ln = g.ln_gamma != nullptr;

  // The tiles fill the 227 KB almost completely, so the launch cannot afford a spare kilobyte of
  // alignment slack: a base that is not 1024-aligned is reported instead of silently overrun.
  if (pad + SMEM_TILES + N_BARS * 8 + 16 + (g.hidden + 3 * g.C) * 4 > g.smem_bytes) {
    if (threadIdx.x == 0) atomicExch(g.status, (int)SMARTMEM_ERR_UNSUPPORTED);
    return;
  }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int NC = g.n_chunks;
  const int k1_last = (g.C - BK) / 16;             // k16 steps of the second k-block of fc1 (C <= 128)
  const int nkb1 = g.C > BK ? 2 : 1;
  const int my_tiles = ((int)g.tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
  const int total = my_tiles * NC;                 // hidden chunks this CTA walks through, over all its tiles

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&a_full[i], 1);
      ptx::mbar_init(&a_empty[i], 1);
      ptx::mbar_init(&s1_full[i], 1);
      ptx::mbar_init(&s1_empty[i], 1);                       // fc2 of the chunk has consumed the buffer (its H)
      ptx::mbar_init(&h_full[i], kGeluWarps);                // H of buffer i written (GELU warps)
      ptx::mbar_init(&out_full[i], 1);
      ptx::mbar_init(&out_empty[i], kOutWarps);
      ptx::mbar_init(&a_ready[i], kNormWarps);
    }
    for (int i = 0; i < NST; ++i) {
      ptx::mbar_init(&w_full[i], 1);
      ptx::mbar_init(&w_empty[i], 1);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmW1);
    ptx::prefetch_tensormap(&tmW2);
  }
  for (int i = threadIdx.x; i < g.hidden; i += kThreads) b1_s[i] = __bfloat162float(g.b1[i]);
  for (int i = threadIdx.x; i < g.C; i += kThreads) b2_s[i] = __bfloat162float(g.b2[i]);
  if (fuse_ln)
    for (int i = threadIdx.x; i < g.C; i += kThreads) {
      reinterpret_cast<__nv_bfloat16*>(ln_s)[i] = g.ln_gamma[i];              // packed bf16: [C] gamma at word 0, [C] beta at word C
      reinterpret_cast<__nv_bfloat16*>(ln_s + g.C)[i] = g.ln_beta[i];
    }
  if (warp == 1) ptx::tmem_alloc(tmem_slot, TMEM_COLS);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                       // everything above (weights' biases included) overlapped the previous kernel's tail
  pdl_launch_dependents();

  // fc1 runs one hidden chunk ahead of fc2 over the CTA's whole chunk sequence, across tile
  // boundaries; each has its own issuing thread.  The weights of both share one ring, filled in
  // the order  W1(0), then for j = 0..total-1: W1(j+1), W2(j).
  if (warp == 0) {
    if (lane == 0) {
      uint32_t ws = 0, wph = 1;
      bool ok = true;
      auto load_a = [&](int ti) {                      // ti: this CTA's ti-th tile
        const int b = ti & 1;
        ok = ok && ptx::mbar_wait_relaxed(&a_empty[b], ((ti >> 1) & 1) ^ 1, abort_flag, g.status);
        if (!ok) return;
        const int t = (int)blockIdx.x + ti * (int)gridDim.x;
        ptx::mbar_expect_tx(&a_full[b], nkb1 * KB_BYTES);
        for (int kb = 0; kb < nkb1; ++kb)
          ptx::tma_load_2d(sA + (b * 2 + kb) * KB_BYTES, &tmA, &a_full[b], kb * BK, t * BM);
      };
      auto load_w1 = [&](int c) {                      // [128 hidden rows] x C, as nkb1 k-blocks
        ok = ok && ptx::mbar_wait_relaxed(&w_empty[ws], wph, abort_flag, g.status);
        if (!ok) return;
        ptx::mbar_expect_tx(&w_full[ws], nkb1 * KB_BYTES);
        for (int kb = 0; kb < nkb1; ++kb) ptx::tma_load_2d(sW + ws * WST_BYTES + kb * KB_BYTES, &tmW1, &w_full[ws], kb * BK, c * HC);
        if (++ws == NST) { ws = 0; wph ^= 1; }
      };
      auto load_w2 = [&](int c) {                      // [C rows] x 128 hidden columns, as 2 k-blocks
        ok = ok && ptx::mbar_wait_relaxed(&w_empty[ws], wph, abort_flag, g.status);
        if (!ok) return;
        ptx::mbar_expect_tx(&w_full[ws], 2 * (uint32_t)g.C * BK * 2);
        for (int kb = 0; kb < 2; ++kb) ptx::tma_load_2d(sW + ws * WST_BYTES + kb * KB_BYTES, &tmW2, &w_full[ws], c * HC + kb * BK, 0);
        if (++ws == NST) { ws = 0; wph ^= 1; }
      };
      if (total > 0) {
        load_a(0);
        load_w1(0);
      }
      int ti = 0, c = 0;
      for (int j = 0; j < total && ok; ++j) {
        if (c == 0 && ti + 1 < my_tiles) load_a(ti + 1);     // the next tile's rows, a whole tile ahead
        const int cn = c + 1 == NC ? 0 : c + 1;
        if (j + 1 < total) load_w1(cn);
        load_w2(c);
        c = cn;
        if (c == 0) ++ti;
      }
    }
  } else if (warp == 1) {
    // fc1 issuer: S1[j & 1] = A W1[chunk j]^T, one chunk ahead of fc2.  Weight ring entry of
    // chunk j's W1: 0 for j = 0, else 2j - 1 (the producer's order above).
    if (lane == 0) {
      const uint32_t idesc1 = ptx::make_idesc_bf16(BM, HC, false, false);
      const uint32_t a_base = ptx::smem_u32(sA), w_base = ptx::smem_u32(sW);
      int it1 = 0, c1 = 0;
      bool ok = true;
      for (int j = 0; j < total && ok; ++j) {
        const uint32_t sb = j & 1, ab = it1 & 1;
        const uint32_t n = j ? 2 * j - 1 : 0, ws = n % NST, wph = (n / NST) & 1;
        if (c1 == 0) ok = ptx::mbar_wait(fuse_ln ? &a_ready[ab] : &a_full[ab], (it1 >> 1) & 1, abort_flag, g.status);
        ok = ok && ptx::mbar_wait(&s1_empty[sb], ((j >> 1) & 1) ^ 1, abort_flag, g.status);
        ok = ok && ptx::mbar_wait(&w_full[ws], wph, abort_flag, g.status);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t d = tmem_base + TM_S1 + sb * HC;
        const uint64_t ad = ptx::make_smem_desc(a_base + ab * 2 * KB_BYTES, 16, 1024);
        const uint64_t bd = ptx::make_smem_desc(w_base + ws * WST_BYTES, 16, 1024);
        issue_kblock(d, ad, bd, idesc1, BK / 16, false);
        if (nkb1 > 1) issue_kblock(d, ad + (KB_BYTES >> 4), bd + (KB_BYTES >> 4), idesc1, k1_last, true);
        ptx::tc_commit(&w_empty[ws]);
        ptx::tc_commit(&s1_full[sb]);
        if (++c1 == NC) {
          ptx::tc_commit(&a_empty[ab]);                 // every fc1 MMA of this tile has been issued
          c1 = 0;
          ++it1;
        }
      }
    }
  } else if (warp == 2 + kGeluWarps + kOutWarps) {
    // fc2 issuer: OUT[tile & 1] += H[j & 1] W2[:, chunk j]^T.  Ring entry of chunk j's W2:
    // 2j + 2, except for the very last chunk, which no W1 load precedes: 2j + 1.
    if (lane == 0) {
      const uint32_t idesc2 = ptx::make_idesc_bf16(BM, g.C, false, false);
      const uint32_t w_base = ptx::smem_u32(sW);
      int it2 = 0, c2 = 0;
      bool ok = true;
      for (int j = 0; j < total && ok; ++j) {
        const uint32_t ob = it2 & 1;
        const uint32_t n = j + 1 < total ? 2 * j + 2 : 2 * j + 1, ws = n % NST, wph = (n / NST) & 1;
        const uint32_t sb = j & 1;
        ok = ptx::mbar_wait(&h_full[sb], (j >> 1) & 1, abort_flag, g.status);
        if (c2 == 0) ok = ok && ptx::mbar_wait(&out_empty[ob], ((it2 >> 1) & 1) ^ 1, abort_flag, g.status);
        ok = ok && ptx::mbar_wait(&w_full[ws], wph, abort_flag, g.status);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t d = tmem_base + TM_OUT + ob * OUT_STRIDE;
        // H chunk: 128 bf16 per lane, written by the GELU warps over the S1 buffer it was computed from --
        // hidden columns 0..63 as 32 packed columns at offset 0, columns 64..127 at offset 64
        const uint32_t a = tmem_base + TM_S1 + sb * HC;
        const uint64_t bd = ptx::make_smem_desc(w_base + ws * WST_BYTES, 16, 1024);
        ptx::tc_mma_bf16_ta(d, a, bd, idesc2, c2 != 0 ? 1u : 0u);
#pragma unroll
        for (int k = 1; k < HC / 16; ++k)               // 16 hidden columns = 8 packed TMEM columns per step
          ptx::tc_mma_bf16_ta(d, a + 8 * k + (k >= 4 ? 32 : 0), bd + (k >> 2) * (KB_BYTES >> 4) + 2 * (k & 3), idesc2, 1u);
        ptx::tc_commit(&w_empty[ws]);
        ptx::tc_commit(&s1_empty[sb]);                  // buffer consumed: fc1 of chunk j + 2 may overwrite it
        if (++c2 == NC) {
          ptx::tc_commit(&out_full[ob]);
          c2 = 0;
          ++it2;
        }
      }
    }
  } else if (warp < 2 + kGeluWarps) {
    // GELU warps: S1 chunk (TMEM, fp32) -> + b1 -> GELU -> bf16 pairs -> the H region of TMEM, where
    // fc2 reads the chunk as its A operand.  H overwrites (half of) the S1 columns it was computed from,
    // so each of the two S1 buffers carries its chunk from fc1 through GELU to fc2 and is handed back to
    // fc1 by fc2's commit; the GELU warps themselves wait for nothing but the next fc1 result.
    const int e = warp - 2, q = warp & 3, hh = e >> 2;   // quadrant, half of the chunk's 128 columns
    bool ok = true;
    int c = 0;
    for (int j = 0; j < total && ok; ++j) {
      const uint32_t sb = j & 1;
      const float4* bb4 = reinterpret_cast<const float4*>(b1_s + c * HC + hh * 64);   // this warp's 64 biases of the chunk: 16-byte broadcast reads
      ok = ptx::mbar_wait(&s1_full[sb], (j >> 1) & 1, abort_flag, g.status);
      if (!ok) break;
      const uint32_t tq = tmem_base + TM_S1 + sb * HC + ((uint32_t)(q * 32) << 16) + hh * 64;
      uint32_t rv[64];
      ptx::tc_fence_after();
      ptx::tmem_ld32(tq, rv);
      ptx::tmem_ld32(tq + 32, rv + 32);
      ptx::tmem_ld_wait();
      uint32_t pk[32];
#pragma unroll
      for (int v = 0; v < 16; ++v) {
        const float4 b4 = bb4[v];
        pk[2 * v] = gelu_tanh_bf16x2(__uint_as_float(rv[4 * v]) + b4.x, __uint_as_float(rv[4 * v + 1]) + b4.y);
        pk[2 * v + 1] = gelu_tanh_bf16x2(__uint_as_float(rv[4 * v + 2]) + b4.z, __uint_as_float(rv[4 * v + 3]) + b4.w);
      }
      // the packed result goes over the first 32 of the 64 columns this warp has just read (it is the only
      // reader and writer of them), so no warp ever waits for fc2 of an earlier chunk
      ptx::tmem_st32(tq, pk);
      ptx::tmem_st_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&h_full[sb]);
      if (++c == NC) c = 0;
    }
  } else if (warp < 2 + kGeluWarps + kOutWarps) {
    // Output warps, one per TMEM lane quadrant: OUT + b2 + residual -> out, a thread per row, in
    // rounds of 32 columns.  They work on one OUT buffer while fc2 of the next tile fills the other.
    const int q = warp & 3;
    const int rounds = g.C / 32;
    bool ok = true;
    for (int ti = 0; ti < my_tiles && ok; ++ti) {
      const uint32_t ob = ti & 1;
      const int t = (int)blockIdx.x + ti * (int)gridDim.x;
      const int row = t * BM + q * 32 + lane;
      const bool row_ok = row < g.M;
      const long long off = (long long)row * g.C;
      ok = ptx::mbar_wait_relaxed(&out_full[ob], (ti >> 1) & 1, abort_flag, g.status, 256);
      if (!ok) break;
      ptx::tc_fence_after();
#pragma unroll 1                                          // (once per tile: a short body beats a long straight line of cold code)
      for (int r = 0; r < rounds; ++r) {
        {
          uint32_t rv[32];
          ptx::tmem_ld32(tmem_base + TM_OUT + ob * OUT_STRIDE + ((uint32_t)(q * 32) << 16) + r * 32, rv);
          uint4 res[4];                                  // the residual's latency overlaps the accumulator load
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            res[v] = make_uint4(0, 0, 0, 0);
            if (g.residual && row_ok) res[v] = *reinterpret_cast<const uint4*>(g.residual + off + r * 32 + v * 8);
          }
          ptx::tmem_ld_wait();
          if (r + 1 == rounds) {                         // the accumulator is in registers: hand the buffer back
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&out_empty[ob]);
          }
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            const uint32_t w[4] = {res[v].x, res[v].y, res[v].z, res[v].w};
            float a8[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 f = bf16x2_to_float2(w[i]);
              const float2 b = *reinterpret_cast<const float2*>(b2_s + r * 32 + v * 8 + 2 * i);
              a8[2 * i] = fmaf(__uint_as_float(rv[v * 8 + 2 * i]), 0.5f, b.x) + f.x;        // the accumulator holds 2 H W2^T
              a8[2 * i + 1] = fmaf(__uint_as_float(rv[v * 8 + 2 * i + 1]), 0.5f, b.y) + f.y;
            }
            uint4 pk;
            pk.x = float2_to_bf16x2(a8[0], a8[1]);
            pk.y = float2_to_bf16x2(a8[2], a8[3]);
            pk.z = float2_to_bf16x2(a8[4], a8[5]);
            pk.w = float2_to_bf16x2(a8[6], a8[7]);
            if (row_ok) *reinterpret_cast<uint4*>(g.out + off + r * 32 + v * 8) = pk;
          }
        }
      }
    }
  } else if (warp >= 3 + kGeluWarps + kOutWarps) {
    // LayerNorm warps: the producer brought the raw rows of the tile into the A buffer (K-major,
    // 128-byte swizzle); normalise them in place, a thread per row, before fc1 reads them.  Two
    // passes over the row in registers (mean, then squared deviations), statistics in fp32.
    if (fuse_ln) {
      const int nw = warp - (3 + kGeluWarps + kOutWarps);
      const float invC = 1.0f / (float)g.C;
      const int nch = g.C / 8;                           // 16-byte chunks per row: 8 or 12
      bool ok = true;
      for (int ti = 0; ti < my_tiles && ok; ++ti) {
        const int b = ti & 1;
        ok = ptx::mbar_wait_relaxed(&a_full[b], (ti >> 1) & 1, abort_flag, g.status, 64);
        if (!ok) break;
        for (int rr = 0; rr < BM / (32 * kNormWarps); ++rr) {
          const int r = (rr * kNormWarps + nw) * 32 + lane;
          uint8_t* row0 = sA + (b * 2) * KB_BYTES + r * 128;
          // Both passes read the row from shared memory with partly unrolled loops instead of keeping it in registers: this code
          // runs once per tile, and a long straight-line body costs more in instruction fetch than the re-read does.
          // One pass over the row for both moments, on data shifted by the row's first element p (d = x - p):
          // mean = p + sum(d) / C, variance = (sum(d^2) - sum(d)^2 / C) / C.  p lies within the row's own spread,
          // so the subtraction of the two sums loses a few bits at most.  Four independent partial sums each.
          const float p = __uint_as_float(*reinterpret_cast<const uint32_t*>(row0 + ((0 ^ (r & 7)) << 4)) << 16);
          float s4[4] = {0.f, 0.f, 0.f, 0.f}, q4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
          for (int ch = 0; ch < nch; ++ch) {
            const uint4 xv = *reinterpret_cast<const uint4*>(row0 + (ch >> 3) * KB_BYTES + (((ch & 7) ^ (r & 7)) << 4));
            const uint32_t w[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 f = bf16x2_to_float2(w[i]);
              const float dx = f.x - p, dy = f.y - p;
              s4[i] += dx + dy;
              q4[i] = fmaf(dy, dy, fmaf(dx, dx, q4[i]));
            }
          }
          const float sd = (s4[0] + s4[1]) + (s4[2] + s4[3]);
          const float mean = fmaf(sd, invC, p);
          const float sq = fmaxf(((q4[0] + q4[1]) + (q4[2] + q4[3])) - sd * sd * invC, 0.f);
          const float rstd = rsqrtf(sq * invC + g.ln_eps);
          const float nmr = -mean * rstd;
#pragma unroll 4
          for (int ch = 0; ch < nch; ++ch) {
            uint4* px = reinterpret_cast<uint4*>(row0 + (ch >> 3) * KB_BYTES + (((ch & 7) ^ (r & 7)) << 4));
            const uint4 xv = *px;
            const uint32_t w[4] = {xv.x, xv.y, xv.z, xv.w};
            // (x - mean) rstd in fp32, rounded to bf16 pairs; the affine part as one packed multiply-add per pair
            const uint4 ga = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(ln_s) + ch * 8);
            const uint4 be = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(ln_s + g.C) + ch * 8);
            const uint32_t gw[4] = {ga.x, ga.y, ga.z, ga.w}, bw[4] = {be.x, be.y, be.z, be.w};
            uint32_t o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 f = bf16x2_to_float2(w[i]);
              const uint32_t t = float2_to_bf16x2(fmaf(f.x, rstd, nmr), fmaf(f.y, rstd, nmr));
              asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(o[i]) : "r"(t), "r"(gw[i]), "r"(bw[i]));
            }
            *px = make_uint4(o[0], o[1], o[2], o[3]);
          }
        }
        ptx::fence_proxy_async();                        // generic-proxy writes -> visible to the MMA's reads
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&a_ready[b]);
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace

bool mlp_fused_supported(long long C, long long hidden) {
  return (C == 64 || C == 96) && hidden >= HC && hidden % HC == 0 && hidden <= 512;
}

int launch_mlp_fused(const void* A, const void* ln_gamma, const void* ln_beta, float ln_eps, const void* W1, const void* b1,
                     const void* W2, const void* b2, const void* residual, void* out, long long M, long long C,
                     long long hidden, cudaStream_t st) {
  if (!mlp_fused_supported(C, hidden) || M < 1 || M >= (1ll << 31) - BM) return SMARTMEM_ERR_UNSUPPORTED;
  const void* ptrs[] = {A, W1, b1, W2, b2, residual, out, ln_gamma, ln_beta};
  if ((ln_gamma == nullptr) != (ln_beta == nullptr)) return SMARTMEM_ERR_INVALID_ARG;
  for (const void* p : ptrs)
    if ((uintptr_t)p & 15) return SMARTMEM_ERR_ALIGNMENT;
  if (!b1 || !b2) return SMARTMEM_ERR_INVALID_ARG;
  CUtensorMap ta, tw1, tw2;
  int rc;
  if ((rc = tc_encode_2d(A, C, M, C, BK, BM, &ta)) != SMARTMEM_OK) return rc;
  if ((rc = tc_encode_2d(W1, C, hidden, C, BK, HC, &tw1)) != SMARTMEM_OK) return rc;
  if ((rc = tc_encode_2d(W2, hidden, C, hidden, BK, (int)C, &tw2)) != SMARTMEM_OK) return rc;
  MlpArgs g;
  memset(&g, 0, sizeof(g));
  g.M = (int)M; g.C = (int)C; g.hidden = (int)hidden; g.n_chunks = (int)(hidden / HC);
  g.tiles = (int)((M + BM - 1) / BM);
  g.b1 = (const __nv_bfloat16*)b1; g.b2 = (const __nv_bfloat16*)b2; g.residual = (const __nv_bfloat16*)residual;
  g.out = (__nv_bfloat16*)out;
  g.ln_gamma = (const __nv_bfloat16*)ln_gamma; g.ln_beta = (const __nv_bfloat16*)ln_beta; g.ln_eps = ln_eps;
  g.status = device_status_ptr();
  if (!g.status) return SMARTMEM_ERR_CUDA;
  const size_t need = (size_t)SMEM_TILES + N_BARS * 8 + 16 + (size_t)(hidden + 3 * C) * 4;
  const size_t smem = need + 1024 <= 232448 ? need + 1024 : 232448;     // alignment slack only while it fits
  if (need > smem) return SMARTMEM_ERR_UNSUPPORTED;
  g.smem_bytes = (uint32_t)smem;
  if (ensure_max_dynamic_smem((const void*)mlp_fused_kernel, 232448) != SMARTMEM_OK) return SMARTMEM_ERR_CUDA;
  profile_tick("mlp_fused", st);
  const unsigned grid = (unsigned)(g.tiles < tc_sm_count() ? g.tiles : tc_sm_count());
  launch_pdl(mlp_fused_kernel, dim3(grid), dim3(kThreads), smem, st, ta, tw1, tw2, g);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

}  // namespace smartmem
