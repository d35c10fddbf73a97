// Fused MLP half of a transformer block on tcgen05:
//
//   out = A + GELU(LN(A) W1^T + b1) W2^T + b2,     A [M, C], W1 [hidden, C], W2 [C, hidden]
//
// for narrow blocks (C in {64, 96}), where the hidden activation [M, hidden] is four times larger
// than everything else the block touches.  Neither the normalised rows nor the hidden tensor leave
// the SM, and A is read from global memory exactly once.
//
// Both weight matrices stay resident in shared memory for the whole kernel (2 x 72 KB at C = 96),
// so the only stream through the SM is the raw rows of A.  LayerNorm is folded into fc1 (see
// tc_tiles.cuh): every CTA scales its copy of W1 by gamma once, the raw rows go to the tensor core
// unchanged, the mean / sigma terms (and b1) ride on one extra k16 step, and the GELU warps multiply
// the accumulator by the row's rstd.  Because the raw rows are still in shared memory, the residual
// is a tensor-core product too: OUT = A I opens the output accumulator of a tile (I: a 32 x 32
// identity tile per 32-column k-block), and fc2 accumulates on top of it.
//
// Per 128-row tile: the producer brings the raw rows in by TMA (double-buffered across tiles), four
// warps take the row statistics (a thread per row); then the kernel walks over chunks of 128 hidden
// columns: fc1 of a chunk accumulates in one of two S1 buffers in TMEM, a set of GELU warps applies rstd
// and GELU on packed bf16 pairs and writes the bf16 chunk into one of two H buffers in TMEM, and fc2
// takes it from there as its A operand (tensor memory).  The S1 buffer goes back to fc1 as soon as the
// GELU warps have read it, the H buffer comes back with fc2's commit, so fc1, GELU and fc2 of
// neighbouring chunks overlap.  There is one output accumulator; the output warps copy it to registers
// and hand it back before they convert and store.
//
// Warp roles: 0 TMA producer, 1 fc1 issuer and TMEM owner, 2-17 GELU (two sets of eight for the even
// and the odd chunks; in a set two warps per TMEM lane quadrant, 64 hidden columns each), 18-21
// output, 22 fc2 issuer (+ the residual / bias product), 23-26 row statistics.  The issuer warps walk
// their loops with all lanes and elect one lane for the tensor-core instructions: with warp-uniform
// control flow the descriptors stay in uniform registers, which roughly halves the cost of issuing a
// product compared with a branch on lane 0.
//
// What bounds it (clock stamps of every hand-off): the fc2 issuer's chain -- per chunk its eight
// products queue behind the seven of fc1 on the one tensor pipe (about 800 cycles), per tile the
// residual / bias products and the wait for the output warps to hand the accumulator back -- and the
// GELU warps (tanh on the special-function unit, 16 elements per clock per SM).  Isolated, the kernel
// runs 17 us at 100 352 rows, 4 us of which are the prologue (144 KB of weights per SM from L2 and the
// fold); back to back with other kernels that prologue overlaps the previous kernel's tail.  An earlier
// version streamed the weights from L2 through a ring for every tile (113 MB of L2 reads per launch,
// against 21 MB now) and normalised the rows in place; with all of its arithmetic compiled out it still
// took 18 us.

#include "gemm_tc.cuh"
#include "ptx.cuh"
#include "tc_tiles.cuh"

namespace smartmem {
namespace {

using ptx::f32x2;

constexpr int BM = 128, KB = 32, HC = 128;         // tile rows, k-block columns (64-byte rows), hidden chunk
constexpr int KBT = BM * KB * 2;                   // one 128 x 32 bf16 block: 8 KB
constexpr int AX_BYTES = BM * 32;                  // the extra k-step of a tile: 128 rows x 16 bf16
constexpr int ID_BYTES = 32 * 64;                  // identity tile
constexpr int kGeluWarps = 16, kOutWarps = 4, kStatWarps = 4, kThreads = 32 * (3 + kGeluWarps + kOutWarps + kStatWarps);
constexpr uint32_t TM_S1 = 0, TM_H = 2 * HC, TM_OUT = 3 * HC, TMEM_COLS = 512;   // S1 x2 (128 columns), H x2 (64 columns of bf16 pairs), OUT (C columns)
constexpr int N_BARS = 18;
constexpr int RSTD_RING = 4;                       // tiles whose rstd may be live at once (statistics run up to two tiles ahead of GELU)

struct MlpArgs {
  int M, C, hidden, n_chunks, tiles;
  uint32_t smem_bytes;
  const __nv_bfloat16 *b1, *b2, *ln_gamma, *ln_beta;
  float ln_eps;
  __nv_bfloat16* out;
  int* status;
};

__host__ __device__ inline size_t mlp_smem_tiles(int C, int hidden) {
  return (size_t)2 * (C / KB) * KBT + (size_t)2 * hidden * C * 2 + 2 * AX_BYTES + (size_t)hidden * 32 + ID_BYTES + (size_t)C * 32;
}
__host__ __device__ inline size_t mlp_smem_need(int C, int hidden) {
  return mlp_smem_tiles(C, hidden) + N_BARS * 8 + 16 + (size_t)(2 * C + RSTD_RING * BM) * 4;
}

// tanh-form GELU (times two, see below) of two pre-activations, evaluated on packed bf16 pairs: the result is stored as
// bf16 anyway, and the packed path costs one conversion, four packed multiply-adds and one
// tanh.approx per PAIR, where the fp32 form costs seven instructions per element.
__device__ __forceinline__ uint32_t gelu_tanh_bf16x2(float a, float b) {
  const uint32_t u = float2_to_bf16x2(a, b);
  constexpr uint32_t C0 = 0x3F4C3F4Cu, C1 = 0x3D123D12u;   // 0.7979, 0.03568
  uint32_t u2, p, in, t, r;
  asm("mul.rn.bf16x2 %0, %1, %1;" : "=r"(u2) : "r"(u));
  asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(p) : "r"(C1), "r"(u2), "r"(C0));
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(in) : "r"(u), "r"(p));
  asm("tanh.approx.bf16x2 %0, %1;" : "=r"(t) : "r"(in));
  // u (1 + tanh) = TWICE the GELU: the factor 1/2 is a power of two, so it commutes with every rounding on the way and is
  // applied for free where the output warps add b2 (one multiply-add instead of one add); the identity tile of the
  // residual product holds 2 for the same reason
  asm("fma.rn.bf16x2 %0, %1, %2, %1;" : "=r"(r) : "r"(u), "r"(t));
  return r;
}

template <int NKB>
__global__ void __launch_bounds__(kThreads, 1)
mlp_fused_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW1,
                 const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ MlpArgs g) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t pad = (1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  constexpr int C = NKB * KB;
  const int NC = g.n_chunks;
  constexpr int A_BYTES = NKB * KBT;                   // a tile's raw rows: NKB k-blocks of 32 columns
  const int W1_KB = g.hidden * 64;                 // one k-block of W1: [hidden rows][64 B]
  constexpr int W2_KB = C * 64;                        // one k-block of W2: [C rows][64 B]
  uint8_t* sA = smem;                              // [2][NKB][8 KB]
  uint8_t* sW1 = sA + 2 * A_BYTES;                 // [NKB][hidden x 64 B]
  uint8_t* sW2 = sW1 + NKB * W1_KB;                // [hidden / 32][C x 64 B]
  uint8_t* sAx = sW2 + (g.hidden / KB) * W2_KB;    // [2][128 rows x 32 B]
  uint8_t* sW1x = sAx + 2 * AX_BYTES;              // [hidden rows x 32 B]
  uint8_t* sId = sW1x + g.hidden * 32;             // [32 rows x 64 B]
  uint8_t* sB2x = sId + ID_BYTES;                  // [C rows x 32 B]: 2 b2 on the positions where the extra k-step's rows hold ones
  uint64_t* bars = reinterpret_cast<uint64_t*>(sB2x + C * 32);
  uint64_t *a_full = bars, *a_empty = bars + 2, *a_ready = bars + 4, *s1_full = bars + 6, *s1_free = bars + 8;
  uint64_t *h_full = bars + 10, *h_empty = bars + 12, *out_full = bars + 14, *out_empty = bars + 15;
  uint64_t *w1_full = bars + 16, *w2_full = bars + 17;

  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + N_BARS);
  int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);
  float* ln_s = reinterpret_cast<float*>(tmem_slot + 4);     // [2][C]: gamma, beta
  float* rstd_s = ln_s + 2 * C;                              // [RSTD_RING][128]

  // The tiles fill the 227 KB almost completely, so the launch cannot afford a spare kilobyte of
  // alignment slack: a base that is not 1024-aligned is reported instead of silently overrun.
  if (pad + mlp_smem_need(C, g.hidden) + 16 > g.smem_bytes) {
    if (threadIdx.x == 0) atomicExch(g.status, (int)SMARTMEM_ERR_UNSUPPORTED);
    return;
  }

  const int tid = threadIdx.x, warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0), lane = tid & 31;   // (warp: provably uniform)
  const int my_tiles = ((int)g.tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
  const int total = my_tiles * NC;                 // hidden chunks this CTA walks through, over all its tiles

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&a_full[i], 1);
      ptx::mbar_init(&a_empty[i], 2);                        // the last fc1 product and the residual product of the tile
      ptx::mbar_init(&a_ready[i], kStatWarps);
    }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&s1_full[i], 1);
      ptx::mbar_init(&s1_free[i], kGeluWarps / 2);           // the chunk's GELU warps have read S1 buffer i
      ptx::mbar_init(&h_full[i], kGeluWarps / 2);            // H buffer i written (by the set of GELU warps that has the chunk)
      ptx::mbar_init(&h_empty[i], 1);                        // fc2 of the chunk has consumed H buffer i
    }
    ptx::mbar_init(out_full, 1);
    ptx::mbar_init(out_empty, kOutWarps);
    ptx::mbar_init(w1_full, 1);
    ptx::mbar_init(w2_full, 1);
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmW1);
    ptx::prefetch_tensormap(&tmW2);
    // the weights: parameters, not produced by the kernel before this one, so they are requested before the dependency wait
    ptx::mbar_expect_tx(w1_full, (uint32_t)g.hidden * (uint32_t)C * 2u);
#pragma unroll 1
    for (int kb = 0; kb < NKB; ++kb)
#pragma unroll 1
      for (int c = 0; c < NC; ++c) ptx::tma_load_2d(sW1 + kb * W1_KB + c * KBT, &tmW1, w1_full, kb * KB, c * HC);
    ptx::mbar_expect_tx(w2_full, (uint32_t)g.hidden * (uint32_t)C * 2u);
#pragma unroll 1
    for (int kb = 0; kb < g.hidden / KB; ++kb) ptx::tma_load_2d(sW2 + kb * W2_KB, &tmW2, w2_full, kb * KB, 0);
  }
#pragma unroll 1
  for (int i = tid; i < C; i += kThreads) {
    ln_s[i] = __bfloat162float(g.ln_gamma[i]);
    ln_s[C + i] = __bfloat162float(g.ln_beta[i]);
    uint4 k0, k1;
    bias_col(2.0f * __bfloat162float(g.b2[i]), k0, k1);     // (the output accumulator holds twice the result)
    *reinterpret_cast<uint4*>(sB2x + plain_off(i, 0)) = k0;
    *reinterpret_cast<uint4*>(sB2x + plain_off(i, 1)) = k1;
  }
#pragma unroll 1
  for (int i = tid; i < (2 * AX_BYTES + ID_BYTES) / 16; i += kThreads) {
    uint8_t* p = i < 2 * AX_BYTES / 16 ? sAx + i * 16 : sId + (i - 2 * AX_BYTES / 16) * 16;
    *reinterpret_cast<uint4*>(p) = make_uint4(0, 0, 0, 0);
  }
  if (warp == 1) ptx::tmem_alloc(tmem_slot, TMEM_COLS);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (warp == 1)                                      // identity: row n has a two in column n
    *reinterpret_cast<uint16_t*>(sId + sw64_off(lane, lane >> 3) + (lane & 7) * 2) = 0x4000u;
  // From here on warp 0 is the producer on its own; the other warps fold gamma into the resident W1 (the column
  // terms c_n and b'_n go into the extra k-step) and meet at a barrier of their own before they take up their
  // roles.  Two threads per weight row (the first and second half of its 16-byte chunks); 2 * hidden and the
  // number of folding threads are multiples of 32, so whole warps take part in every round.
  bool w_ok = true;
  if (warp != 0) {
    w_ok = __all_sync(0xFFFFFFFFu, ptx::mbar_wait(w1_full, 0, abort_flag, g.status) ? 1 : 0) != 0;
    if (w_ok) {
      const int nch = C / 8;
#pragma unroll 1
      for (int t2 = tid - 32; t2 < 2 * g.hidden; t2 += kThreads - 32) {
        const int row = t2 >> 1, half = t2 & 1;
        float csum = 0.f, bsum = half ? 0.f : __bfloat162float(g.b1[row]);
        float bsum2 = 0.f;
#pragma unroll 2
        for (int ci = half * (nch / 2); ci < (half + 1) * (nch / 2); ++ci) {     // chunk ci of the row: k-block ci / 4, chunk ci % 4
          uint4* p = reinterpret_cast<uint4*>(sW1 + (ci >> 2) * W1_KB + sw64_off(row, ci & 3));
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
          *reinterpret_cast<uint4*>(sW1x + plain_off(row, 0)) = k0;
          *reinterpret_cast<uint4*>(sW1x + plain_off(row, 1)) = k1;
        }
      }
    }
    ptx::fence_proxy_async();                         // the rewritten weights, identity and zeros -> visible to the MMAs
    asm volatile("bar.sync 1, %0;" ::"n"(kThreads - 32) : "memory");
  }
  pdl_wait();                       // everything above touched parameters only: it overlaps the previous kernel's tail
  pdl_launch_dependents();

  if (warp == 0) {
    // producer: the raw rows of the CTA's tiles, one tile ahead
    if (lane == 0) {
      bool ok = true;
#pragma unroll 1
      for (int ti = 0; ti < my_tiles && ok; ++ti) {
        const int b = ti & 1;
        ok = ptx::mbar_wait_relaxed(&a_empty[b], ((ti >> 1) & 1) ^ 1, abort_flag, g.status);
        if (!ok) break;
        const int t = (int)blockIdx.x + ti * (int)gridDim.x;
        ptx::mbar_expect_tx(&a_full[b], (uint32_t)A_BYTES);
#pragma unroll 1
        for (int kb = 0; kb < NKB; ++kb) ptx::tma_load_2d(sA + b * A_BYTES + kb * KBT, &tmA, &a_full[b], kb * KB, t * BM);
      }
    }
  } else if (warp == 1) {
    // fc1 issuer: S1[j & 1] = A W1'[chunk j]^T + the extra k-step, as soon as the GELU warps have read the buffer
    if (w_ok) {                                         // (the whole warp walks the loop; one elected lane issues)
      const uint32_t idesc1 = ptx::make_idesc_bf16(BM, HC, false, false);
      const uint32_t a_base = ptx::smem_u32(sA), w_base = ptx::smem_u32(sW1), ax_base = ptx::smem_u32(sAx);
      const uint32_t wx_base = ptx::smem_u32(sW1x);
      int it1 = 0, c1 = 0;
      bool ok = true;
#pragma unroll 1
      for (int j = 0; j < total && ok; ++j) {
        const uint32_t ab = it1 & 1, sb = j & 1, ph = (j >> 1) & 1;
        if (c1 == 0) ok = ptx::mbar_wait(&a_ready[ab], (it1 >> 1) & 1, abort_flag, g.status);
        ok = ok && ptx::mbar_wait(&s1_free[sb], ph ^ 1, abort_flag, g.status);
        ok = __all_sync(0xFFFFFFFFu, ok ? 1 : 0) != 0;
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t d = tmem_base + TM_S1 + sb * HC;
        const uint64_t ad = desc_sw64(a_base + ab * A_BYTES);
        const uint64_t bd = desc_sw64(w_base + c1 * KBT);
        const bool last = c1 + 1 == NC;
        if (ptx::elect_one()) {
#pragma unroll
          for (int kb = 0; kb < NKB; ++kb) {
            ptx::tc_mma_bf16(d, ad + kb * (KBT >> 4), bd + kb * (W1_KB >> 4), idesc1, kb ? 1u : 0u);
            ptx::tc_mma_bf16(d, ad + kb * (KBT >> 4) + 2, bd + kb * (W1_KB >> 4) + 2, idesc1, 1u);
          }
          ptx::tc_mma_bf16(d, desc_plain(ax_base + ab * AX_BYTES), desc_plain(wx_base + c1 * (HC * 32)), idesc1, 1u);
          ptx::tc_commit(&s1_full[sb]);
          if (last) ptx::tc_commit(&a_empty[ab]);       // every fc1 product of this tile has been issued
        }
        __syncwarp();
        if (last) {
          c1 = 0;
          ++it1;
        } else {
          ++c1;
        }
      }
    }
  } else if (warp == 2 + kGeluWarps + kOutWarps) {
    // fc2 issuer: at the first chunk of a tile OUT = A (2 I) + 2 b2; then OUT += H[j & 1] W2[:, chunk j]^T
    if (w_ok) {
      const uint32_t idesc2 = ptx::make_idesc_bf16(BM, C, false, false);
      const uint32_t idesc_id = ptx::make_idesc_bf16(BM, 32, false, false);
      const uint32_t w_base = ptx::smem_u32(sW2), a_base = ptx::smem_u32(sA);
      const uint64_t idd = desc_sw64(ptx::smem_u32(sId)), b2d = desc_plain(ptx::smem_u32(sB2x));
      const uint32_t ax_base = ptx::smem_u32(sAx);
      const uint32_t d = tmem_base + TM_OUT;
      int it2 = 0, c2 = 0;
      bool ok = __all_sync(0xFFFFFFFFu, ptx::mbar_wait(w2_full, 0, abort_flag, g.status) ? 1 : 0) != 0;
#pragma unroll 1
      for (int j = 0; j < total && ok; ++j) {
        const uint32_t sb = j & 1, ph = (j >> 1) & 1;
        ok = ptx::mbar_wait(&h_full[sb], ph, abort_flag, g.status);
        if (c2 == 0) ok = ok && ptx::mbar_wait(out_empty, (it2 & 1) ^ 1, abort_flag, g.status);
        ok = __all_sync(0xFFFFFFFFu, ok ? 1 : 0) != 0;
        if (!ok) break;
        ptx::tc_fence_after();
        // H chunk: 128 hidden columns as 64 columns of bf16 pairs
        const uint32_t a = tmem_base + TM_H + sb * (HC / 2);
        const uint64_t bd = desc_sw64(w_base + c2 * 4 * W2_KB);
        const uint64_t ad = desc_sw64(a_base + (it2 & 1) * A_BYTES);
        const bool first = c2 == 0, last = c2 + 1 == NC;
        if (ptx::elect_one()) {
          if (first) {
#pragma unroll
            for (int kb = 0; kb < NKB; ++kb) {
              ptx::tc_mma_bf16(d + kb * KB, ad + kb * (KBT >> 4), idd, idesc_id, 0u);
              ptx::tc_mma_bf16(d + kb * KB, ad + kb * (KBT >> 4) + 2, idd + 2, idesc_id, 1u);
            }
            ptx::tc_mma_bf16(d, desc_plain(ax_base + (it2 & 1) * AX_BYTES), b2d, idesc2, 1u);   // + 2 b2
            ptx::tc_commit(&a_empty[it2 & 1]);          // the raw rows have had their last reader
          }
#pragma unroll
          for (int k = 0; k < HC / 16; ++k)             // 16 hidden columns = 8 packed TMEM columns per step
            ptx::tc_mma_bf16_ta(d, a + 8 * k, bd + (k >> 1) * (W2_KB >> 4) + 2 * (k & 1), idesc2, 1u);
          ptx::tc_commit(&h_empty[sb]);                 // H buffer consumed: GELU of chunk j + 2 may overwrite it
          if (last) ptx::tc_commit(out_full);
        }
        __syncwarp();
        if (last) {
          c2 = 0;
          ++it2;
        } else {
          ++c2;
        }
      }
    }
  } else if (warp < 2 + kGeluWarps) {
    // GELU warps: S1 chunk (TMEM, fp32) -> x rstd -> GELU -> bf16 pairs -> an H buffer in TMEM, where fc2 reads
    // the chunk as its A operand.  Two sets of eight warps take the even and the odd chunks (S1 and H buffer
    // = set), so that one set's tensor-memory loads and stores overlap the other's arithmetic (tanh on the
    // special-function unit is what bounds them); in a set, two warps per TMEM lane quadrant with 64 hidden
    // columns each, in two rounds of 32.  The S1 buffer goes back to fc1 as soon as the set has read it; the H
    // buffer comes back from fc2's commit.
    const int e = warp - 2, set = e >> 3, q = warp & 3, hh = (e & 7) >> 2;
    bool ok = w_ok;
    int c = set, ti = 0;
    while (c >= NC) { c -= NC; ++ti; }
    uint32_t ph = 0;
    const uint32_t lane_q = (uint32_t)(q * 32) << 16;
    const uint32_t ts = tmem_base + TM_S1 + set * HC + lane_q + hh * 64;
    const uint32_t th = tmem_base + TM_H + set * (HC / 2) + lane_q + hh * 32;
#pragma unroll 1
    for (int j = set; j < total && ok; j += 2) {
      ok = ptx::mbar_wait(&s1_full[set], ph, abort_flag, g.status);
      if (!ok) break;
      const float rstd = rstd_s[(ti & (RSTD_RING - 1)) * BM + q * 32 + lane];
      const f32x2 r2 = ptx::pack2(rstd, rstd);
      ptx::tc_fence_after();
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {
        uint32_t rv[32];
        ptx::tmem_ld32(ts + h2 * 32, rv);
        ptx::tmem_ld_wait();
        if (h2 == 1) {                                   // S1 is in registers: fc1 of chunk j + 2 may overwrite the buffer
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&s1_free[set]);
        }
        uint32_t pk[16];
#pragma unroll
        for (int v = 0; v < 16; ++v) {
          float xa, xb;
          ptx::unpack2(ptx::mul2(ptx::pack2(__uint_as_float(rv[2 * v]), __uint_as_float(rv[2 * v + 1])), r2), xa, xb);
          pk[v] = gelu_tanh_bf16x2(xa, xb);
        }
        if (h2 == 0) {                                   // fc2 of chunk j - 2 has read the H buffer
          ok = ptx::mbar_wait(&h_empty[set], ph ^ 1, abort_flag, g.status);
          if (!ok) break;
          ptx::tc_fence_after();
        }
        ptx::tmem_st16(th + h2 * 16, pk);
      }
      if (!ok) break;
      ptx::tmem_st_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&h_full[set]);
      c += 2;
      while (c >= NC) { c -= NC; ++ti; }
      ph ^= 1;
    }
  } else if (warp < 2 + kGeluWarps + kOutWarps) {
    // Output warps, one per TMEM lane quadrant: OUT / 2 + b2 -> out, a thread per row, in rounds of 32
    // columns.  They work on one OUT buffer while the products of the next tile fill the other.
    const int q = warp & 3;
    const int rounds = C / 32;
    const f32x2 half2 = ptx::pack2(0.5f, 0.5f);
    const bool wide_store = (reinterpret_cast<uintptr_t>(g.out) & 31) == 0;
    bool ok = w_ok;
#pragma unroll 1
    for (int ti = 0; ti < my_tiles && ok; ++ti) {
      const int t = (int)blockIdx.x + ti * (int)gridDim.x;
      const int row = t * BM + q * 32 + lane;
      const bool row_ok = row < g.M;
      const long long off = (long long)row * C;
      ok = ptx::mbar_wait_relaxed(out_full, ti & 1, abort_flag, g.status, 256);
      if (!ok) break;
      ptx::tc_fence_after();
#pragma unroll 1                                          // (once per tile: a short body beats a long straight line of cold code)
      for (int r = 0; r < rounds; ++r) {
        uint32_t rv[32];
        ptx::tmem_ld32(tmem_base + TM_OUT + ((uint32_t)(q * 32) << 16) + r * 32, rv);
        ptx::tmem_ld_wait();
        if (r + 1 == rounds) {                         // the accumulator is in registers: hand the buffer back
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(out_empty);
        }
        uint4 o_prev = make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint32_t o[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {                // the accumulator holds 2 (A + H W2^T + b2)
            float xa, xb;
            ptx::unpack2(ptx::mul2(ptx::pack2(__uint_as_float(rv[v * 8 + 2 * i]), __uint_as_float(rv[v * 8 + 2 * i + 1])), half2), xa, xb);
            o[i] = float2_to_bf16x2(xa, xb);
          }
          // whole 32-byte sectors per store when the output is aligned for it (rows are 128 or 192 bytes apart)
          if (wide_store) {
            if (v & 1) {
              if (row_ok) ptx::st_global_v8(g.out + off + r * 32 + (v - 1) * 8, o_prev, make_uint4(o[0], o[1], o[2], o[3]));
            } else {
              o_prev = make_uint4(o[0], o[1], o[2], o[3]);
            }
          } else if (row_ok) *reinterpret_cast<uint4*>(g.out + off + r * 32 + v * 8) = make_uint4(o[0], o[1], o[2], o[3]);
        }
      }
    }
  } else if (warp >= 3 + kGeluWarps + kOutWarps) {
    // Statistics warps: the producer brought the raw rows of the tile into the A buffer (K-major, 64-byte
    // swizzle); a thread per row takes mean and variance in two passes over shared memory (fp32) and writes
    // the row's side of the extra k-step.  The loops are only partly unrolled: this code runs once per tile,
    // and fetching its instructions costs as much as executing them.
    const int r = (warp - (3 + kGeluWarps + kOutWarps)) * 32 + lane;
    const float invC = 1.0f / (float)C;
    const int nch = C / 8;                               // 16-byte chunks per row: 8 or 12
    bool ok = w_ok;
#pragma unroll 1
    for (int ti = 0; ti < my_tiles && ok; ++ti) {
      const int b = ti & 1;
      ok = ptx::mbar_wait_relaxed(&a_full[b], (ti >> 1) & 1, abort_flag, g.status, 64);
      if (!ok) break;
      const uint8_t* rowp = sA + b * A_BYTES;
      f32x2 s2[2] = {0ull, 0ull};
#pragma unroll 4
      for (int ch = 0; ch < nch; ++ch) {
        const uint4 xv = *reinterpret_cast<const uint4*>(rowp + (ch >> 2) * KBT + sw64_off(r, ch & 3));
        const uint32_t x4[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
        for (int e = 0; e < 4; ++e)
          s2[e & 1] = ptx::add2(s2[e & 1], ptx::pack2(__uint_as_float(x4[e] << 16), __uint_as_float(x4[e] & 0xFFFF0000u)));
      }
      float a0, a1, a2, a3;
      ptx::unpack2(s2[0], a0, a1);
      ptx::unpack2(s2[1], a2, a3);
      const float mean = ((a0 + a1) + (a2 + a3)) * invC;
      const f32x2 nm2 = ptx::pack2(-mean, -mean);
      f32x2 q2[2] = {0ull, 0ull};
#pragma unroll 4
      for (int ch = 0; ch < nch; ++ch) {
        const uint4 xv = *reinterpret_cast<const uint4*>(rowp + (ch >> 2) * KBT + sw64_off(r, ch & 3));
        const uint32_t x4[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const f32x2 d2 = ptx::add2(ptx::pack2(__uint_as_float(x4[e] << 16), __uint_as_float(x4[e] & 0xFFFF0000u)), nm2);
          q2[e & 1] = ptx::fma2(d2, d2, q2[e & 1]);
        }
      }
      ptx::unpack2(q2[0], a0, a1);
      ptx::unpack2(q2[1], a2, a3);
      const float var = ((a0 + a1) + (a2 + a3)) * invC + g.ln_eps;
      const float rstd = rsqrtf(var);
      uint4 k0, k1;
      extra_row(-mean, var * rstd, k0, k1);              // sigma = var / sqrt(var)
      rstd_s[(ti & (RSTD_RING - 1)) * BM + r] = rstd;
      *reinterpret_cast<uint4*>(sAx + b * AX_BYTES + plain_off(r, 0)) = k0;
      *reinterpret_cast<uint4*>(sAx + b * AX_BYTES + plain_off(r, 1)) = k1;
      ptx::fence_proxy_async();                          // generic-proxy writes -> visible to the MMA's reads
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&a_ready[b]);
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
  if (!((C == 64 || C == 96) && hidden >= HC && hidden % HC == 0 && hidden <= 512)) return false;
  return mlp_smem_need((int)C, (int)hidden) + 16 <= 232448;
}

int launch_mlp_fused(const void* A, const void* ln_gamma, const void* ln_beta, float ln_eps, const void* W1, const void* b1,
                     const void* W2, const void* b2, void* out, long long M, long long C, long long hidden,
                     cudaStream_t st) {
  if (!mlp_fused_supported(C, hidden) || M < 1 || M >= (1ll << 31) - BM) return SMARTMEM_ERR_UNSUPPORTED;
  const void* ptrs[] = {A, W1, b1, W2, b2, out, ln_gamma, ln_beta};
  for (const void* p : ptrs) {
    if (!p) return SMARTMEM_ERR_INVALID_ARG;
    if ((uintptr_t)p & 15) return SMARTMEM_ERR_ALIGNMENT;
  }
  CUtensorMap ta, tw1, tw2;
  int rc;
  {
    const long long dims[2] = {C, M}, strides[1] = {C};
    const int box[2] = {KB, BM};
    if ((rc = tc_encode_nd_sw64(A, 2, dims, strides, box, &ta)) != SMARTMEM_OK) return rc;
  }
  {
    const long long dims[2] = {C, hidden}, strides[1] = {C};
    const int box[2] = {KB, HC};
    if ((rc = tc_encode_nd_sw64(W1, 2, dims, strides, box, &tw1)) != SMARTMEM_OK) return rc;
  }
  {
    const long long dims[2] = {hidden, C}, strides[1] = {hidden};
    const int box[2] = {KB, (int)C};
    if ((rc = tc_encode_nd_sw64(W2, 2, dims, strides, box, &tw2)) != SMARTMEM_OK) return rc;
  }
  MlpArgs g;
  memset(&g, 0, sizeof(g));
  g.M = (int)M; g.C = (int)C; g.hidden = (int)hidden; g.n_chunks = (int)(hidden / HC);
  g.tiles = (int)((M + BM - 1) / BM);
  g.b1 = (const __nv_bfloat16*)b1; g.b2 = (const __nv_bfloat16*)b2;
  g.out = (__nv_bfloat16*)out;
  g.ln_gamma = (const __nv_bfloat16*)ln_gamma; g.ln_beta = (const __nv_bfloat16*)ln_beta; g.ln_eps = ln_eps;
  g.status = device_status_ptr();
  if (!g.status) return SMARTMEM_ERR_CUDA;
  const size_t need = mlp_smem_need((int)C, (int)hidden) + 16;
  const size_t smem = need + 1024 <= 232448 ? need + 1024 : 232448;     // alignment slack only while it fits
  g.smem_bytes = (uint32_t)smem;
  auto* kern = C == 96 ? mlp_fused_kernel<3> : mlp_fused_kernel<2>;
  if (ensure_max_dynamic_smem((const void*)kern, 232448) != SMARTMEM_OK) return SMARTMEM_ERR_CUDA;
  profile_tick("mlp_fused", st);
  const unsigned grid = (unsigned)(g.tiles < tc_sm_count() ? g.tiles : tc_sm_count());
  launch_pdl(kern, dim3(grid), dim3(kThreads), smem, st, ta, tw1, tw2, g);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

}  // namespace smartmem
