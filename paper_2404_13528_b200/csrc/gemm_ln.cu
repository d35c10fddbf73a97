// LayerNorm o row-gather o linear in one kernel, for narrow rows (K = C in {64, 96}):
//
//   out[m, :] = LN(X[src(m), :]) W^T + b,      X rows of K elements, W [N, K], N = nsub * 96
//
// `src` is the composed index map of the layout operators that sit between the producer of X and
// this linear layer (cyclic shift and window partition in a Swin block): the rows are gathered as
// they are loaded, so neither the normalised nor the re-ordered tensor is ever written.
//
// What makes the narrow case different from a general GEMM: a 128-row tile has only K/16 <= 6 MMA
// k-steps of work per 96 output columns, so the cost of a tile is everything around the MMAs.
// Hence
//   * the whole weight matrix stays in shared memory for the life of the CTA (72 KB at N = 288),
//   * an A tile is produced once and used by all nsub column sub-tiles,
//   * the A producers are eight ordinary warps, two threads per row: they load the row from global
//     memory (through the index map), normalise it in registers (two-pass statistics in fp32) and
//     write it in the K-major 128-byte-swizzled operand layout; the next tile's rows are already in
//     flight while the current ones are normalised,
//   * accumulators form a ring of five 96-column TMEM buffers, handed to eight epilogue warps
//     sub-tile by sub-tile (bias, bf16, swizzled per-quadrant staging, asynchronous TMA stores).
//
// Warp roles: 0 idle after set-up (thread 0 fetches the weights by TMA, once), 1 MMA issuer + TMEM
// owner, 2-9 epilogue, 10-17 A producers.
#include "gemm_tc.cuh"
#include "ptx.cuh"


namespace smartmem {
namespace {

constexpr int BM = 128, BK = 64, BN = 96;
constexpr int KB_BYTES = BM * BK * 2;              // one 128 x 64 bf16 operand block: 16 KB
constexpr int A_BYTES = 2 * KB_BYTES;              // an A tile: two k-blocks
constexpr int NA = 3, NACC = 5;                    // A ring depth, accumulator ring depth
constexpr int kEpiWarps = 8, kProdWarps = 8, kThreads = 32 * (2 + kEpiWarps + kProdWarps);
constexpr int ST_A = 32 * 128, ST_B = 32 * 64;      // staging of a quadrant's 32 x 96 sub-tile: columns 0-63 (128-byte
                                                   // swizzle) and 64-95 (64-byte swizzle), the two boxes its TMA stores read
constexpr int ST_BYTES = ST_A + ST_B;              // x 2 buffers x 4 quadrants
constexpr uint32_t TMEM_COLS = 512;

struct LnGemmArgs {
  int M, N, K, nsub, tiles, has_map, has_ln;
  float eps;
  uint32_t smem_bytes;
  const __nv_bfloat16 *x, *gamma, *beta, *bias;
  __nv_bfloat16* out;
  int* status;
  DevMap rowmap;
};

template <int KDIM>
__global__ void __launch_bounds__(kThreads, 1)
gemm_ln_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmOA,
               const __grid_constant__ CUtensorMap tmOB, const __grid_constant__ LnGemmArgs g) {
  constexpr int NH = KDIM / 16;                    // 16-byte chunks per half row (one thread's share)
  constexpr int NKB = KDIM > BK ? 2 : 1;
  constexpr int K1_STEPS = (KDIM - BK) / 16;       // k16 steps of the second k-block
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t pad = (1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  const int b_kb_bytes = g.N * 128;                // one k-block of the weights: N rows x 128 bytes
  uint8_t* sA = smem;                              // [NA][2 k-blocks][16 KB]
  uint8_t* sB = sA + NA * A_BYTES;                 // [NKB][N rows x 128 B]
  uint8_t* qstage_base = sB + NKB * b_kb_bytes;    // [4 quadrants][2 buffers][ST_BYTES]; 1024-aligned (N is a multiple of 96)
  float* bias_s = reinterpret_cast<float*>(qstage_base + 4 * 2 * ST_BYTES);   // [N]
  float* ln_s = bias_s + g.N;                      // [2][K]: gamma, beta
  uint64_t* bars = reinterpret_cast<uint64_t*>(ln_s + 2 * KDIM);
  uint64_t *a_full = bars, *a_empty = bars + NA, *acc_full = bars + 2 * NA, *acc_empty = acc_full + NACC;
  uint64_t* b_full = acc_empty + NACC;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(b_full + 1);
  int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);

  if (pad + (uint32_t)(reinterpret_cast<uint8_t*>(tmem_slot + 4) - smem) > g.smem_bytes) {
    if (threadIdx.x == 0) atomicExch(g.status, (int)SMARTMEM_ERR_UNSUPPORTED);
    return;
  }

  const int warp = __shfl_sync(0xFFFFFFFFu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // (warp: provably uniform)
  const int nsub = g.nsub;
  const int my_tiles = ((int)g.tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NA; ++i) {
      ptx::mbar_init(&a_full[i], kProdWarps);
      ptx::mbar_init(&a_empty[i], 1);
    }
    for (int i = 0; i < NACC; ++i) {
      ptx::mbar_init(&acc_full[i], 1);
      ptx::mbar_init(&acc_empty[i], kEpiWarps);
    }
    ptx::mbar_init(b_full, 1);
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
    // the weights do not depend on the kernel before this one: fetch them right away
    ptx::prefetch_tensormap(&tmW);
    ptx::prefetch_tensormap(&tmOA);
    ptx::prefetch_tensormap(&tmOB);
    ptx::mbar_expect_tx(b_full, (uint32_t)(NKB * nsub * BN * 128));
    for (int kb = 0; kb < NKB; ++kb)
      for (int j = 0; j < nsub; ++j)
        ptx::tma_load_2d(sB + kb * b_kb_bytes + j * (BN * 128), &tmW, b_full, kb * BK, j * BN);
  }
  if (warp == 1) ptx::tmem_alloc(tmem_slot, TMEM_COLS);
  for (int i = threadIdx.x; i < g.N; i += kThreads) bias_s[i] = g.bias ? __bfloat162float(g.bias[i]) : 0.f;
  if (g.has_ln)
    for (int i = threadIdx.x; i < KDIM; i += kThreads) {
      reinterpret_cast<__nv_bfloat16*>(ln_s)[i] = g.gamma[i];                 // packed bf16: gamma at word 0, beta at word KDIM
      reinterpret_cast<__nv_bfloat16*>(ln_s + KDIM)[i] = g.beta[i];
    }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                       // everything above depends on parameters only
  pdl_launch_dependents();

  if (warp == 1) {
    // ---- MMA issuer: the whole warp walks the loop, one elected lane issues (warp-uniform control flow keeps the
    // descriptors in uniform registers) -----------------------------------------------------------
    {
      const uint32_t idesc = ptx::make_idesc_bf16(BM, BN, false, false);
      const uint32_t a_base = ptx::smem_u32(sA), b_base = ptx::smem_u32(sB);
      bool ok = __all_sync(0xFFFFFFFFu, ptx::mbar_wait(b_full, 0, abort_flag, g.status) ? 1 : 0) != 0;
      uint32_t ab = 0, aph = 0, buf = 0, cph = 1;     // A ring position / phase, accumulator ring position / phase
      for (int ti = 0; ti < my_tiles && ok; ++ti) {
        ok = __all_sync(0xFFFFFFFFu, ptx::mbar_wait(&a_full[ab], aph, abort_flag, g.status) ? 1 : 0) != 0;
        const uint64_t ad = ptx::make_smem_desc(a_base + ab * A_BYTES, 16, 1024);
        for (int j = 0; j < nsub && ok; ++j) {
          ok = __all_sync(0xFFFFFFFFu, ptx::mbar_wait(&acc_empty[buf], cph, abort_flag, g.status) ? 1 : 0) != 0;
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t d = tmem_base + buf * BN;
          const uint64_t bd = ptx::make_smem_desc(b_base + j * (BN * 128), 16, 1024);
          const bool last = j + 1 == nsub;
          if (ptx::elect_one()) {
            ptx::tc_mma_bf16(d, ad, bd, idesc, 0u);
#pragma unroll
            for (int k = 1; k < BK / 16; ++k) ptx::tc_mma_bf16(d, ad + 2 * k, bd + 2 * k, idesc, 1u);
            if (NKB > 1) {
              const uint64_t ad1 = ad + (KB_BYTES >> 4), bd1 = bd + (uint64_t)(b_kb_bytes >> 4);
#pragma unroll
              for (int k = 0; k < K1_STEPS; ++k) ptx::tc_mma_bf16(d, ad1 + 2 * k, bd1 + 2 * k, idesc, 1u);
            }
            ptx::tc_commit(&acc_full[buf]);
            if (last) ptx::tc_commit(&a_empty[ab]);   // every MMA that reads this A tile has been issued
          }
          __syncwarp();
          if (++buf == NACC) { buf = 0; cph ^= 1; }
        }
        if (++ab == NA) { ab = 0; aph ^= 1; }
      }
    }
  } else if (warp >= 2 && warp < 2 + kEpiWarps) {
    // ---- epilogue: warp (quadrant q, column half) owns 32 rows x 48 columns of a sub-tile ----
    // The quadrant's two warps stage their 32 x 96 block in shared memory and one thread hands it
    // to two TMA stores, which drain in the background: the warps go on with the next sub-tile
    // instead of waiting on the store path (all SMs write in bursts that would otherwise stall them).
    const int e = warp - 2, q = warp & 3, half = e >> 2;
    uint8_t* qstage = qstage_base + q * (2 * ST_BYTES);
    const bool elected = half == 0 && lane == 0;
    bool ok = true;
    uint32_t buf = 0, cph = 0, cnt = 0;
    for (int ti = 0; ti < my_tiles && ok; ++ti) {
      const int t = (int)blockIdx.x + ti * (int)gridDim.x;
      for (int j = 0; j < nsub; ++j, ++cnt) {
        uint8_t* stA = qstage + (cnt & 1) * ST_BYTES;
        uint8_t* stB = stA + ST_A;
        // the store issued from this staging buffer two sub-tiles ago must have read it
        if (elected) ptx::bulk_wait_group_read<1>();
        asm volatile("bar.sync %0, 64;" ::"r"(1 + q) : "memory");
        ok = ptx::mbar_wait(&acc_full[buf], cph, abort_flag, g.status);
        if (ok) {
          uint32_t rv[48];
          ptx::tc_fence_after();
          const uint32_t ta = tmem_base + buf * BN + ((uint32_t)(q * 32) << 16) + half * 48;
          ptx::tmem_ld32(ta, rv);
          ptx::tmem_ld16(ta + 32, rv + 32);
          ptx::tmem_ld_wait();
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&acc_empty[buf]);
          const float* bb = bias_s + j * BN + half * 48;
#pragma unroll
          for (int v = 0; v < 6; ++v) {
            const float4 b0 = *reinterpret_cast<const float4*>(bb + v * 8), b1 = *reinterpret_cast<const float4*>(bb + v * 8 + 4);
            uint4 pk;
            pk.x = float2_to_bf16x2(__uint_as_float(rv[v * 8 + 0]) + b0.x, __uint_as_float(rv[v * 8 + 1]) + b0.y);
            pk.y = float2_to_bf16x2(__uint_as_float(rv[v * 8 + 2]) + b0.z, __uint_as_float(rv[v * 8 + 3]) + b0.w);
            pk.z = float2_to_bf16x2(__uint_as_float(rv[v * 8 + 4]) + b1.x, __uint_as_float(rv[v * 8 + 5]) + b1.y);
            pk.w = float2_to_bf16x2(__uint_as_float(rv[v * 8 + 6]) + b1.z, __uint_as_float(rv[v * 8 + 7]) + b1.w);
            const int ch = half * 6 + v;                 // 16-byte chunk of the 192-byte row
            if (ch < 8) *reinterpret_cast<uint4*>(stA + lane * 128 + ((ch ^ (lane & 7)) << 4)) = pk;
            else *reinterpret_cast<uint4*>(stB + lane * 64 + (((ch - 8) ^ ((lane >> 1) & 3)) << 4)) = pk;
          }
          ptx::fence_proxy_async();                      // generic-proxy writes -> visible to the TMA store
        }
        // the quadrant's four warps meet (and leave together if one of them gave up waiting)
        uint32_t gave_up;
        asm volatile(
            "{\n\t.reg .pred pin, pout;\n\t"
            "setp.ne.u32 pin, %2, 0;\n\t"
            "bar.red.or.pred pout, %1, 64, pin;\n\t"
            "selp.u32 %0, 1, 0, pout;\n\t}"
            : "=r"(gave_up)
            : "r"(1 + q), "r"(ok ? 0u : 1u)
            : "memory");
        if (gave_up) { ok = false; break; }
        if (elected) {                                  // rows past M are clipped by the tensor map
          ptx::tma_store_2d(&tmOA, stA, j * BN, t * BM + q * 32);
          ptx::tma_store_2d(&tmOB, stB, j * BN + 64, t * BM + q * 32);
          ptx::bulk_commit_group();
        }
        if (++buf == NACC) { buf = 0; cph ^= 1; }
      }
    }
    if (elected) ptx::bulk_wait_group<0>();              // the CTA's shared memory must outlive its stores
  } else if (warp >= 2 + kEpiWarps) {
    // ---- A producers: two threads per row (lane pair), 16 rows per warp --------------------------
    const int pw = warp - (2 + kEpiWarps), hh = lane & 1;
    const int r = pw * 16 + (lane >> 1);               // row inside the tile
    const float invK = 1.0f / (float)KDIM;
    auto load_row = [&](int ti, uint4* x) {
      const int row = ((int)blockIdx.x + ti * (int)gridDim.x) * BM + r;
      long long off = 0;
      if (hh == 0 && row < g.M) off = g.has_map ? devmap_eval_unrolled(g.rowmap, (uint32_t)row) : (long long)row * KDIM;
      off = __shfl_sync(0xFFFFFFFFu, off, lane & ~1);
      const uint4* src = reinterpret_cast<const uint4*>(g.x + off) + hh * NH;
#pragma unroll
      for (int c = 0; c < NH; ++c) x[c] = row < g.M ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
    };
    uint4 cur[NH], nxt[NH];
    if (my_tiles > 0) load_row(0, cur);
    bool ok = true;
    uint32_t ab = 0, aph = 1;
    for (int ti = 0; ti < my_tiles && ok; ++ti) {
      if (ti + 1 < my_tiles) load_row(ti + 1, nxt);    // in flight while this tile is normalised
      if (g.has_ln) {
        // one pass for both moments on data shifted by the row's first element p (d = x - p): mean = p + sum(d) / K,
        // variance = (sum(d^2) - sum(d)^2 / K) / K; p lies within the row's own spread, so the subtraction of the
        // two sums loses a few bits at most.  The two threads of a row share p and add their partial sums.
        const float p = __shfl_sync(0xFFFFFFFFu, __uint_as_float(cur[0].x << 16), lane & ~1);
        float s4[4] = {0.f, 0.f, 0.f, 0.f}, q4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c = 0; c < NH; ++c) {
          const uint32_t w[4] = {cur[c].x, cur[c].y, cur[c].z, cur[c].w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 f = bf16x2_to_float2(w[i]);
            const float dx = f.x - p, dy = f.y - p;
            s4[i] += dx + dy;
            q4[i] = fmaf(dy, dy, fmaf(dx, dx, q4[i]));
          }
        }
        float sd = (s4[0] + s4[1]) + (s4[2] + s4[3]);
        float sq = (q4[0] + q4[1]) + (q4[2] + q4[3]);
        sd += __shfl_xor_sync(0xFFFFFFFFu, sd, 1);
        sq += __shfl_xor_sync(0xFFFFFFFFu, sq, 1);
        const float mean = fmaf(sd, invK, p);
        sq = fmaxf(sq - sd * sd * invK, 0.f);
        const float rstd = rsqrtf(sq * invK + g.eps);
        const float nmr = -mean * rstd;
        // (x - mean) rstd in fp32, rounded to bf16 pairs; the affine part as one packed multiply-add per pair
#pragma unroll
        for (int c = 0; c < NH; ++c) {
          const uint32_t w[4] = {cur[c].x, cur[c].y, cur[c].z, cur[c].w};
          uint32_t o[4];
          const int col = (hh * NH + c) * 8;
          const uint4 ga = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(ln_s) + col);
          const uint4 be = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(ln_s + KDIM) + col);
          const uint32_t gw[4] = {ga.x, ga.y, ga.z, ga.w}, bw[4] = {be.x, be.y, be.z, be.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 f = bf16x2_to_float2(w[i]);
            const uint32_t t = float2_to_bf16x2(fmaf(f.x, rstd, nmr), fmaf(f.y, rstd, nmr));
            asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(o[i]) : "r"(t), "r"(gw[i]), "r"(bw[i]));
          }
          cur[c] = make_uint4(o[0], o[1], o[2], o[3]);
        }
      }
      ok = ptx::mbar_wait_relaxed(&a_empty[ab], aph, abort_flag, g.status, 32);
      if (!ok) break;
      uint8_t* row0 = sA + ab * A_BYTES + r * 128;
#pragma unroll
      for (int c = 0; c < NH; ++c) {
        const int ci = hh * NH + c;                    // chunk of the row: k-block ci / 8, swizzled slot (ci % 8) ^ (r % 8)
        *reinterpret_cast<uint4*>(row0 + (ci >> 3) * KB_BYTES + (((ci & 7) ^ (r & 7)) << 4)) = cur[c];
      }
      ptx::fence_proxy_async();                        // generic-proxy writes -> visible to the MMA's reads
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&a_full[ab]);
      if (++ab == NA) { ab = 0; aph ^= 1; }
#pragma unroll
      for (int c = 0; c < NH; ++c) cur[c] = nxt[c];
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

template <int KDIM>
int launch_t(const CUtensorMap& tw, const CUtensorMap& toa, const CUtensorMap& tob, LnGemmArgs& g, size_t smem, cudaStream_t st) {
  if (ensure_max_dynamic_smem((const void*)gemm_ln_kernel<KDIM>, 232448) != SMARTMEM_OK) return SMARTMEM_ERR_CUDA;
  const unsigned grid = (unsigned)(g.tiles < tc_sm_count() ? g.tiles : tc_sm_count());
  if (launch_pdl(gemm_ln_kernel<KDIM>, dim3(grid), dim3(kThreads), smem, st, tw, toa, tob, g) != cudaSuccess) return SMARTMEM_ERR_CUDA;
  count_launch();
  return SMARTMEM_OK;
}

}  // namespace

bool gemm_ln_supported(long long N, long long K) {
  return (K == 64 || K == 96) && N % BN == 0 && N / BN >= 1 && N / BN <= 3;
}

int launch_gemm_ln(const void* X, const DevMap* rowmap, const void* gamma, const void* beta, float eps, const void* W,
                   const void* bias, void* out, long long M, long long N, long long K, cudaStream_t st) {
  if (!gemm_ln_supported(N, K) || M < 1 || M >= (1ll << 31) - BM) return SMARTMEM_ERR_UNSUPPORTED;
  const void* ptrs[] = {X, gamma, beta, W, bias, out};
  for (const void* p : ptrs)
    if ((uintptr_t)p & 15) return SMARTMEM_ERR_ALIGNMENT;
  if ((gamma == nullptr) != (beta == nullptr)) return SMARTMEM_ERR_INVALID_ARG;
  CUtensorMap tw, toa, tob;
  int rc = tc_encode_2d(W, K, N, K, BK, BN, &tw);
  if (rc != SMARTMEM_OK) return rc;
  if ((rc = tc_encode_2d(out, N, M, N, 64, 32, &toa)) != SMARTMEM_OK) return rc;         // columns 0-63 of a sub-tile
  if ((rc = tc_encode_2d_sw64(out, N, M, N, 32, 32, &tob)) != SMARTMEM_OK) return rc;    // columns 64-95
  LnGemmArgs g;
  memset(&g, 0, sizeof(g));
  g.M = (int)M; g.N = (int)N; g.K = (int)K; g.nsub = (int)(N / BN);
  g.tiles = (int)((M + BM - 1) / BM);
  g.has_map = rowmap ? 1 : 0;
  if (rowmap) g.rowmap = *rowmap;
  g.has_ln = gamma ? 1 : 0;
  g.eps = eps;
  g.x = (const __nv_bfloat16*)X; g.gamma = (const __nv_bfloat16*)gamma; g.beta = (const __nv_bfloat16*)beta;
  g.bias = (const __nv_bfloat16*)bias; g.out = (__nv_bfloat16*)out;
  g.status = device_status_ptr();
  if (!g.status) return SMARTMEM_ERR_CUDA;
  const int nkb = K > BK ? 2 : 1;
  const size_t need = (size_t)NA * A_BYTES + (size_t)nkb * N * 128 + 4 * 2 * ST_BYTES + (size_t)(N + 2 * K) * 4 +
                      (2 * NA + 2 * NACC + 1) * 8 + 16;
  const size_t smem = need + 1024 <= 232448 ? need + 1024 : 232448;
  if (need > smem) return SMARTMEM_ERR_UNSUPPORTED;
  g.smem_bytes = (uint32_t)smem;
  profile_tick("gemm_ln", st);
  return K == 96 ? launch_t<96>(tw, toa, tob, g, smem, st) : launch_t<64>(tw, toa, tob, g, smem, st);
}

}  // namespace smartmem
