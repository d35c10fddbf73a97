// Fused MLP half of a transformer block on tcgen05:
//
//   out = residual + GELU(A W1^T + b1) W2^T + b2,        A [M, C], W1 [hidden, C], W2 [C, hidden]
//
// for narrow blocks (C <= 128), where the hidden activation [M, hidden] is four times larger than
// everything else the block touches.  The hidden tensor never leaves the SM: per 128-row tile the
// kernel walks over chunks of 128 hidden columns; fc1 of a chunk accumulates in TMEM, the epilogue
// warps apply bias + GELU and write the chunk as bf16 straight into shared memory in the K-major
// 128-byte-swizzled operand layout, and fc2 consumes it from there as its A operand while fc1 of
// the next chunk is already running (two TMEM buffers for fc1, one accumulator for fc2).
//
// Warp roles: warp 0 TMA producer (A tile double-buffered across tiles, weights streamed through a
// ring: they stay L2-resident), warp 1 MMA issuer + TMEM owner, warps 2-17 epilogue.
#include "gemm_tc.cuh"
#include "ptx.cuh"

#ifdef MLP_EXP_TIMING
__device__ long long g_mlp_dbg[8192];
#define DBG(slot) do { if (blockIdx.x == 0) g_mlp_dbg[(slot)] = clock64(); } while (0)
extern "C" __attribute__((visibility("default"))) int smartmem_debug_read(long long* host, int n) {
  return (int)cudaMemcpyFromSymbol(host, g_mlp_dbg, sizeof(long long) * n);
}
#else
#define DBG(slot) do { } while (0)
#endif

namespace smartmem {
namespace {

constexpr int BM = 128, BK = 64, HC = 128;         // tile rows, k-block, hidden chunk
constexpr int KB_BYTES = BM * BK * 2;              // one 128 x 64 bf16 operand block: 16 KB
constexpr int NST = 3;                             // weight ring stages; one stage = both k-blocks of a chunk's W1 or W2
constexpr int WST_BYTES = 2 * KB_BYTES;
constexpr int kEpiWarps = 16, kThreads = 64 + 32 * kEpiWarps;
constexpr uint32_t TM_S1 = 0, TM_OUT = 256, TMEM_COLS = 512;

struct MlpArgs {
  int M, C, hidden, n_chunks, tiles;
  const __nv_bfloat16 *b1, *b2, *residual;
  __nv_bfloat16* out;
  int* status;
};

__device__ __forceinline__ float gelu_tanh(float u) {
  const float u2 = u * u;
  const float inner = u * fmaf(0.0356774081f, u2, 0.7978845608f);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(inner));
  const float h = 0.5f * u;
  return fmaf(h, t, h);
}

__global__ void __launch_bounds__(kThreads, 1)
mlp_fused_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW1,
                 const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ MlpArgs g) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  uint8_t* sA = smem;                              // [2 k-blocks][16 KB]
  uint8_t* sH = sA + 2 * KB_BYTES;                 // [2 bufs][2 k-blocks][16 KB]
  uint8_t* sW = sH + 4 * KB_BYTES;                 // [NST][2 k-blocks][16 KB]
  uint64_t* bars = reinterpret_cast<uint64_t*>(sW + NST * WST_BYTES);
  uint64_t *a_full = bars, *a_empty = bars + 2, *w_full = bars + 4, *w_empty = w_full + NST;
  uint64_t *s1_full = w_empty + NST, *s1_empty = s1_full + 2, *h_full = s1_empty + 2, *h_empty = h_full + 2;
  uint64_t *out_full = h_empty + 2, *out_empty = out_full + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(out_empty + 1);
  int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);
  uint8_t* qstage_base = reinterpret_cast<uint8_t*>(tmem_slot + 4);
  float* b1_s = reinterpret_cast<float*>(qstage_base + 4 * 32 * (g.C == 128 ? 256 : g.C * 2 + 16));   // [hidden]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int NC = g.n_chunks;
  const int k1_last = (g.C - BK + 15) / 16;        // k16 steps of the second k-block of fc1 (C <= 128)
  const int nkb1 = g.C > BK ? 2 : 1;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&a_full[i], 1);
      ptx::mbar_init(&a_empty[i], 1);
      ptx::mbar_init(&s1_full[i], 1);
      ptx::mbar_init(&s1_empty[i], kEpiWarps);
      ptx::mbar_init(&h_full[i], kEpiWarps);
      ptx::mbar_init(&h_empty[i], 1);
    }
    for (int i = 0; i < NST; ++i) {
      ptx::mbar_init(&w_full[i], 1);
      ptx::mbar_init(&w_empty[i], 1);
    }
    ptx::mbar_init(out_full, 1);
    ptx::mbar_init(out_empty, kEpiWarps);
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
  if (warp == 1) ptx::tmem_alloc(tmem_slot, TMEM_COLS);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t wcnt = 0, it = 0;
      bool ok = true;
      auto load_w1 = [&](int c) {                      // [128 hidden rows] x C, as nkb1 k-blocks
        const int s = wcnt % NST;
        ok = ok && ptx::mbar_wait(&w_empty[s], ((wcnt / NST) & 1) ^ 1, abort_flag, g.status);
        if (!ok) return;
        ptx::mbar_expect_tx(&w_full[s], nkb1 * KB_BYTES);
        for (int kb = 0; kb < nkb1; ++kb) ptx::tma_load_2d(sW + s * WST_BYTES + kb * KB_BYTES, &tmW1, &w_full[s], kb * BK, c * HC);
        ++wcnt;
      };
      auto load_w2 = [&](int c) {                      // [C rows] x 128 hidden columns, as 2 k-blocks
        const int s = wcnt % NST;
        ok = ok && ptx::mbar_wait(&w_empty[s], ((wcnt / NST) & 1) ^ 1, abort_flag, g.status);
        if (!ok) return;
        ptx::mbar_expect_tx(&w_full[s], 2 * (uint32_t)g.C * BK * 2);
        for (int kb = 0; kb < 2; ++kb) ptx::tma_load_2d(sW + s * WST_BYTES + kb * KB_BYTES, &tmW2, &w_full[s], c * HC + kb * BK, 0);
        ++wcnt;
      };
      for (uint32_t t = blockIdx.x; t < (uint32_t)g.tiles && ok; t += gridDim.x, ++it) {
        ok = ptx::mbar_wait(&a_empty[0], (it & 1) ^ 1, abort_flag, g.status);
        if (!ok) break;
        ptx::mbar_expect_tx(&a_full[0], nkb1 * KB_BYTES);
        for (int kb = 0; kb < nkb1; ++kb)
          ptx::tma_load_2d(sA + kb * KB_BYTES, &tmA, &a_full[0], kb * BK, (int)t * BM);
        // weights in the order the MMA warp consumes them
        load_w1(0);
        for (int c = 0; c < NC && ok; ++c) {
          if (c + 1 < NC) load_w1(c + 1);
          load_w2(c);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc1 = ptx::make_idesc_bf16(BM, HC, false, false);
      const uint32_t idesc2 = ptx::make_idesc_bf16(BM, g.C, false, false);
      uint32_t wcnt = 0, it = 0, s1cnt = 0, hcnt = 0;
      bool ok = true;
      for (uint32_t t = blockIdx.x; t < (uint32_t)g.tiles && ok; t += gridDim.x, ++it) {
        ok = ptx::mbar_wait(&a_full[0], it & 1, abort_flag, g.status);
        if (!ok) break;
        auto fc1 = [&]() {                              // S1[buf] = A W1[chunk]^T
          const uint32_t sb = s1cnt & 1;
          ok = ok && ptx::mbar_wait(&s1_empty[sb], ((s1cnt >> 1) & 1) ^ 1, abort_flag, g.status);
          if (ok) {
            const int s = wcnt % NST;
            ok = ptx::mbar_wait(&w_full[s], (wcnt / NST) & 1, abort_flag, g.status);
            if (ok) {
              ptx::tc_fence_after();
              for (int kb = 0; kb < nkb1; ++kb) {
                const uint32_t a0 = ptx::smem_u32(sA + kb * KB_BYTES), b0 = ptx::smem_u32(sW + s * WST_BYTES + kb * KB_BYTES);
                const int ks = kb == 0 ? (g.C < BK ? g.C / 16 : BK / 16) : k1_last;
                for (int k = 0; k < ks; ++k)
                  ptx::tc_mma_bf16(tmem_base + TM_S1 + sb * HC, ptx::make_smem_desc(a0 + k * 32, 16, 1024),
                                   ptx::make_smem_desc(b0 + k * 32, 16, 1024), idesc1, (kb | k) ? 1u : 0u);
              }
              ptx::tc_commit(&w_empty[s]);
              ++wcnt;
            }
          }
          if (ok) ptx::tc_commit(&s1_full[sb]);
          ++s1cnt;
        };
        auto fc2 = [&](int c) {                         // OUT += H[chunk] W2[:, chunk]^T
          const uint32_t hb = hcnt & 1;
          ok = ok && ptx::mbar_wait(&h_full[hb], (hcnt >> 1) & 1, abort_flag, g.status);
          if (ok && c == 0) ok = ptx::mbar_wait(out_empty, (it & 1) ^ 1, abort_flag, g.status);
          if (ok) {
            const int s = wcnt % NST;
            ok = ptx::mbar_wait(&w_full[s], (wcnt / NST) & 1, abort_flag, g.status);
            if (ok) {
              ptx::tc_fence_after();
              for (int kb = 0; kb < 2; ++kb) {
                const uint32_t a0 = ptx::smem_u32(sH + (hb * 2 + kb) * KB_BYTES), b0 = ptx::smem_u32(sW + s * WST_BYTES + kb * KB_BYTES);
                for (int k = 0; k < BK / 16; ++k)
                  ptx::tc_mma_bf16(tmem_base + TM_OUT, ptx::make_smem_desc(a0 + k * 32, 16, 1024),
                                   ptx::make_smem_desc(b0 + k * 32, 16, 1024), idesc2, (c | kb | k) ? 1u : 0u);
              }
              ptx::tc_commit(&w_empty[s]);
              ++wcnt;
            }
          }
          if (ok) ptx::tc_commit(&h_empty[hb]);
          ++hcnt;
        };
        fc1();
        for (int c = 0; c < NC && ok; ++c) {
          if (c + 1 < NC) fc1();
          if (c + 1 == NC && ok) ptx::tc_commit(&a_empty[0]);   // every fc1 MMA of this tile has been issued
          fc2(c);
        }
        if (ok) ptx::tc_commit(out_full);
      }
    }
  } else {
    const int e = warp - 2, q = warp & 3, grp = e >> 2;
    const int QROW = g.C == 128 ? 256 : g.C * 2 + 16;     // C = 128: no room left for the pad
    uint8_t* qstage = qstage_base + q * (32 * QROW);
    uint32_t it = 0, s1cnt = 0, hcnt = 0;
    bool ok = true;
    for (uint32_t t = blockIdx.x; t < (uint32_t)g.tiles && ok; t += gridDim.x, ++it) {
      const int r_tile = q * 32 + lane;                  // row inside the tile = TMEM lane
      const int row = (int)t * BM + r_tile;
      const bool row_ok = row < g.M;
      for (int c = 0; c < NC && ok; ++c, ++s1cnt, ++hcnt) {
        const uint32_t sb = s1cnt & 1, hb = hcnt & 1;
        float bb[32];                                    // this warp's 32 biases of the chunk, fetched before the wait
#pragma unroll
        for (int v = 0; v < 8; ++v) {
          const float4 b4 = *reinterpret_cast<const float4*>(b1_s + c * HC + grp * 32 + v * 4);
          bb[v * 4 + 0] = b4.x; bb[v * 4 + 1] = b4.y; bb[v * 4 + 2] = b4.z; bb[v * 4 + 3] = b4.w;
        }
        ok = ptx::mbar_wait(&s1_full[sb], (s1cnt >> 1) & 1, abort_flag, g.status);
        if (!ok) break;
        ok = ptx::mbar_wait(&h_empty[hb], ((hcnt >> 1) & 1) ^ 1, abort_flag, g.status);   // fc2 done with this buffer
        if (!ok) break;
        ptx::tc_fence_after();
        uint32_t rv[32];
        ptx::tmem_ld32(tmem_base + TM_S1 + sb * HC + ((uint32_t)(q * 32) << 16) + grp * 32, rv);
        ptx::tmem_ld_wait();
        float acc[32];
#pragma unroll
#ifdef MLP_EXP_NOGELU
        for (int j = 0; j < 32; ++j) acc[j] = __uint_as_float(rv[j]) + bb[j];
#else
        for (int j = 0; j < 32; ++j) acc[j] = gelu_tanh(__uint_as_float(rv[j]) + bb[j]);
#endif
        // chunk columns grp*32 .. +31 -> k-block (grp >> 1), 16-byte chunks ((grp & 1) * 4 + v) ^ (row & 7)
        uint8_t* hrow = sH + (hb * 2 + (grp >> 1)) * KB_BYTES + r_tile * 128;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint4 pk;
          pk.x = float2_to_bf16x2(acc[v * 8 + 0], acc[v * 8 + 1]);
          pk.y = float2_to_bf16x2(acc[v * 8 + 2], acc[v * 8 + 3]);
          pk.z = float2_to_bf16x2(acc[v * 8 + 4], acc[v * 8 + 5]);
          pk.w = float2_to_bf16x2(acc[v * 8 + 6], acc[v * 8 + 7]);
          *reinterpret_cast<uint4*>(hrow + ((((grp & 1) * 4 + v) ^ (r_tile & 7)) << 4)) = pk;
        }
        ptx::fence_proxy_async();                        // make the generic-proxy writes visible to the MMA
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          ptx::mbar_arrive(&h_full[hb]);
          ptx::mbar_arrive(&s1_empty[sb]);
        }
      }
      if (!ok) break;
      // ---- final epilogue of the tile: OUT + b2 + residual -> out ------------------------------
      const int CG = g.C / 4;                            // columns per warp: 16, 24 or 32
      const int c0 = grp * CG;
      const long long off = (long long)row * g.C;
      uint4 res[4];
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        res[v] = make_uint4(0, 0, 0, 0);
        if (g.residual && row_ok && v * 8 < CG) res[v] = *reinterpret_cast<const uint4*>(g.residual + off + c0 + v * 8);
      }
      ok = ptx::mbar_wait(out_full, it & 1, abort_flag, g.status);
      if (!ok) break;
      ptx::tc_fence_after();
      {
        uint32_t rv[32];
        const uint32_t ta = tmem_base + TM_OUT + ((uint32_t)(q * 32) << 16) + c0;
        if (CG == 32) ptx::tmem_ld32(ta, rv);
        else {
          ptx::tmem_ld16(ta, rv);
          if (CG == 24) ptx::tmem_ld8(ta + 16, rv + 16);
        }
        ptx::tmem_ld_wait();
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          if (v * 8 < CG) {
            float a8[8], bb[8];
            ElemIO<__nv_bfloat16>::load(g.b2 + c0 + v * 8, bb);
            const uint32_t w[4] = {res[v].x, res[v].y, res[v].z, res[v].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float2 f = bf16x2_to_float2(w[j]);
              a8[2 * j] = __uint_as_float(rv[v * 8 + 2 * j]) + bb[2 * j] + f.x;
              a8[2 * j + 1] = __uint_as_float(rv[v * 8 + 2 * j + 1]) + bb[2 * j + 1] + f.y;
            }
            uint4 pk;
            pk.x = float2_to_bf16x2(a8[0], a8[1]);
            pk.y = float2_to_bf16x2(a8[2], a8[3]);
            pk.z = float2_to_bf16x2(a8[4], a8[5]);
            pk.w = float2_to_bf16x2(a8[6], a8[7]);
            *reinterpret_cast<uint4*>(qstage + lane * QROW + (c0 + v * 8) * 2) = pk;
          }
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(out_empty);
      // the four warps of the quadrant have filled a 32 x C staging tile: store whole rows
      asm volatile("bar.sync %0, 128;" ::"r"(1 + q) : "memory");
      const int VR = g.C / 8, tq = grp * 32 + lane;
      for (int v = tq; v < 32 * VR; v += 128) {
        const int rr = v / VR, seg = v - rr * VR;
        const int grow = (int)t * BM + q * 32 + rr;
        if (grow < g.M)
          *reinterpret_cast<uint4*>(g.out + (long long)grow * g.C + seg * 8) =
              *reinterpret_cast<const uint4*>(qstage + rr * QROW + seg * 16);
      }
      asm volatile("bar.sync %0, 128;" ::"r"(1 + q) : "memory");
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
  return (C == 64 || C == 96) && hidden >= HC && hidden % HC == 0 && hidden <= 1024;
}

int launch_mlp_fused(const void* A, const void* W1, const void* b1, const void* W2, const void* b2, const void* residual,
                     void* out, long long M, long long C, long long hidden, cudaStream_t st) {
  if (!mlp_fused_supported(C, hidden) || M < 1 || M >= (1ll << 31) - BM) return SMARTMEM_ERR_UNSUPPORTED;
  const void* ptrs[] = {A, W1, b1, W2, b2, residual, out};
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
  g.status = device_status_ptr();
  if (!g.status) return SMARTMEM_ERR_CUDA;
  const size_t smem = 1024 + (2 + 4 + 2 * NST) * KB_BYTES + (8 + 2 * NST + 6) * 8 + 16 + 4 * 32 * (C == 128 ? 256 : C * 2 + 16) +
                      (size_t)hidden * 4;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(mlp_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448) != cudaSuccess)
      return SMARTMEM_ERR_CUDA;
    configured = true;
  }
  profile_tick("mlp_fused", st);
  const unsigned grid = (unsigned)(g.tiles < tc_sm_count() ? g.tiles : tc_sm_count());
  mlp_fused_kernel<<<grid, kThreads, smem, st>>>(ta, tw1, tw2, g);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

}  // namespace smartmem
