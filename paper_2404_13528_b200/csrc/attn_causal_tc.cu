// Causal attention (prefill, head dimension 128) on the tcgen05 tensor cores.
//
// One CTA = 128 query positions of one head.  K and V stream through shared memory in tiles of
// 64 keys (TMA, double buffered); S = Q K^T and O += P V are tcgen05.mma with the accumulators in
// TMEM (two S buffers, one O: 256 columns); four softmax warps own one query row per thread (the TMEM lane),
// so row maxima and sums need no shuffles.  P goes back to the tensor core through tensor memory: it is
// written as bf16 pairs over the S buffer it was computed from and read by the second MMA as its A
// operand; V is consumed as it lies in memory ([key, d] rows) through the MN-major operand mode, so no
// transpose of V exists anywhere.  The running maximum is only
// refreshed when it grows by more than 2^8 (then O and the running sum are rescaled), which keeps
// the TMEM read-modify-write of O off the common path.
//
// The 64-key tiles keep a CTA at 96 KB of shared memory and 256 TMEM columns, so TWO CTAs share an
// SM: while one is in its softmax (which is bound by the exponential unit) the other one's MMAs
// run, which a single CTA with one softmax group could not overlap.
//
// q, k, v are addressed as TMA boxes inside the buffer the QKV GEMM wrote ([B*S, 3*H*D], head split
// eliminated) or inside materialised [B, H, S, D] tensors (explicit variant); the output tile is
// stored at column h*D of [B*S, H*D] (head merge eliminated) or into [B, H, S, D].
#include "attn.cuh"
#include "gemm_tc.cuh"
#include "ptx.cuh"


namespace smartmem {
namespace {

constexpr int BQ = 128, BKV = 64, D = 128;
constexpr int KB = 128 * 64 * 2;                      // one 128 x 64 bf16 block (Q, P)
constexpr int KBK = BKV * 64 * 2;                     // one 64 x 64 bf16 block (K, V)
constexpr uint32_t TM_S = 0, TM_O = 128, TMEM_COLS = 256;   // two S buffers of 64 columns, O of 128: two CTAs share an SM's 512
constexpr int kThreads = 192;
constexpr float kRescaleThreshold = 8.0f;             // log2 units

struct TcAttnArgs {
  int S, heads, batch, n_qt;
  int q_col0, k_col0, v_col0, col_per_head;           // TMA column of (operand, head): col0 + h * col_per_head
  long long row_per_batch, row_per_head;              // TMA row of (b, h, t): b * row_per_batch + h * row_per_head + t
  __nv_bfloat16* out;
  long long o_sn, o_sh, o_st;
  float scale_log2;
  uint32_t smem_bytes;
  int* status;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(kThreads, 2)
causal_attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      const __grid_constant__ CUtensorMap tmV, const __grid_constant__ TcAttnArgs g) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t pad = (1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  uint8_t* sQ = smem;                                  // [2 k-blocks][16 KB]
  uint8_t* sK = sQ + 2 * KB;                           // [2 stages][2 k-blocks][8 KB]
  uint8_t* sV = sK + 4 * KBK;                          // [2 stages][2 d-chunks][8 KB]
  uint64_t* bars = reinterpret_cast<uint64_t*>(sV + 4 * KBK);
  uint64_t *q_full = bars, *k_full = bars + 1, *k_empty = bars + 3, *v_full = bars + 5, *v_empty = bars + 7;
  uint64_t *s_full = bars + 9, *s_empty = bars + 11, *p_full = bars + 13, *p_empty = bars + 14, *o_done = bars + 15;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);

  if (pad + 2 * KB + 8 * KBK + 16 * 8 + 16 > g.smem_bytes) {
    if (threadIdx.x == 0) atomicExch(g.status, (int)SMARTMEM_ERR_UNSUPPORTED);
    return;
  }
  const int warp = __shfl_sync(0xFFFFFFFFu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // (warp: provably uniform)
  // heaviest units (last query tiles) first
  const int bh_count = g.batch * g.heads;
  const int qt = g.n_qt - 1 - (int)(blockIdx.x / bh_count);
  const int bh = (int)(blockIdx.x % bh_count);
  const int b = bh / g.heads, h = bh - b * g.heads;
  const int n_kv = min(2 * (qt + 1), (g.S + BKV - 1) / BKV);   // 64-key blocks up to and including the diagonal
  const long long row_base = (long long)b * g.row_per_batch + (long long)h * g.row_per_head;

  if (threadIdx.x == 0) {
    ptx::mbar_init(q_full, 1);
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&k_full[i], 1);
      ptx::mbar_init(&k_empty[i], 1);
      ptx::mbar_init(&v_full[i], 1);
      ptx::mbar_init(&v_empty[i], 1);
      ptx::mbar_init(&s_full[i], 1);
      ptx::mbar_init(&s_empty[i], 1);                 // P(j) lives in S buffer j & 1: freed by the commit of P V (j)
    }
    ptx::mbar_init(p_full, 4);
    ptx::mbar_init(p_empty, 1);
    ptx::mbar_init(o_done, 1);
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(&tmQ);
    ptx::prefetch_tensormap(&tmK);
    ptx::prefetch_tensormap(&tmV);
  }
  if (warp == 1) ptx::tmem_alloc(tmem_slot, TMEM_COLS);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                       // the set-up above overlapped the previous kernel's tail
  pdl_launch_dependents();

  if (warp == 0) {
    if (lane == 0) {
      const int qc = g.q_col0 + h * g.col_per_head, kc = g.k_col0 + h * g.col_per_head, vc = g.v_col0 + h * g.col_per_head;
      ptx::mbar_expect_tx(q_full, 2 * KB);
      for (int kb = 0; kb < 2; ++kb) ptx::tma_load_2d(sQ + kb * KB, &tmQ, q_full, qc + kb * 64, (int)(row_base + qt * BQ));
      bool ok = true;
      for (int j = 0; j < n_kv && ok; ++j) {
        const int s = j & 1;
        const uint32_t ph = (j >> 1) & 1;
        const int krow = (int)(row_base + (long long)j * BKV);
        ok = ptx::mbar_wait(&k_empty[s], ph ^ 1, abort_flag, g.status);
        if (!ok) break;
        ptx::mbar_expect_tx(&k_full[s], 2 * KBK);
        for (int kb = 0; kb < 2; ++kb) ptx::tma_load_2d(sK + (s * 2 + kb) * KBK, &tmK, &k_full[s], kc + kb * 64, krow);
        ok = ptx::mbar_wait(&v_empty[s], ph ^ 1, abort_flag, g.status);
        if (!ok) break;
        ptx::mbar_expect_tx(&v_full[s], 2 * KBK);
        for (int dc = 0; dc < 2; ++dc) ptx::tma_load_2d(sV + (s * 2 + dc) * KBK, &tmV, &v_full[s], vc + dc * 64, krow);
      }
    }
  } else if (warp == 1) {
    // the whole warp walks the issue loop and an elected lane issues: warp-uniform control flow keeps the
    // descriptors in uniform registers
    {
      const uint32_t idesc_s = ptx::make_idesc_bf16(BQ, BKV, false, false);
      const uint32_t idesc_pv = ptx::make_idesc_bf16(BQ, D, false, true);      // V: MN-major B operand
      bool ok = __all_sync(0xFFFFFFFFu, ptx::mbar_wait(q_full, 0, abort_flag, g.status) ? 1 : 0) != 0;
      auto issue_s = [&](int j) {
        const int s = j & 1;
        const uint32_t ph = (j >> 1) & 1;
        ok = ok && ptx::mbar_wait(&s_empty[s], ph ^ 1, abort_flag, g.status);
        ok = ok && ptx::mbar_wait(&k_full[s], ph, abort_flag, g.status);
        ok = __all_sync(0xFFFFFFFFu, ok ? 1 : 0) != 0;
        if (!ok) return;
        ptx::tc_fence_after();
        if (ptx::elect_one()) {
#pragma unroll
          for (int kb = 0; kb < 2; ++kb) {
            const uint64_t ad = ptx::make_smem_desc(ptx::smem_u32(sQ + kb * KB), 16, 1024);
            const uint64_t bd = ptx::make_smem_desc(ptx::smem_u32(sK + (s * 2 + kb) * KBK), 16, 1024);
#pragma unroll
            for (int k = 0; k < 4; ++k)                 // a k16 step moves both start addresses by 32 bytes
              ptx::tc_mma_bf16(tmem_base + TM_S + s * BKV, ad + 2 * k, bd + 2 * k, idesc_s, (kb | k) ? 1u : 0u);
          }
          ptx::tc_commit(&k_empty[s]);
          ptx::tc_commit(&s_full[s]);
        }
        __syncwarp();
      };
      auto issue_pv = [&](int j) {
        const int s = j & 1;
        ok = ok && ptx::mbar_wait(p_full, j & 1, abort_flag, g.status);
        ok = ok && ptx::mbar_wait(&v_full[s], (j >> 1) & 1, abort_flag, g.status);
        ok = __all_sync(0xFFFFFFFFu, ok ? 1 : 0) != 0;
        if (!ok) return;
        ptx::tc_fence_after();
        const uint32_t v0 = ptx::smem_u32(sV + s * 2 * KBK);
        const uint64_t vd = ptx::make_smem_desc(v0, KBK, 1024);
        const uint32_t pa = tmem_base + TM_S + s * BKV;  // P(j): bf16 pairs over the first 32 columns of the S buffer it came from
        if (ptx::elect_one()) {
#pragma unroll
          for (int ks = 0; ks < BKV / 16; ++ks)        // 16 keys per step: P +8 packed columns, V +16 rows of 128 bytes; the two 64-wide d-chunks are KBK apart
            ptx::tc_mma_bf16_ta(tmem_base + TM_O, pa + 8 * ks, vd + (2048 >> 4) * ks, idesc_pv, (j | ks) ? 1u : 0u);
          ptx::tc_commit(&v_empty[s]);
          ptx::tc_commit(&s_empty[s]);
          ptx::tc_commit(p_empty);
        }
        __syncwarp();
      };
      issue_s(0);
      for (int j = 0; j < n_kv && ok; ++j) {
        if (j + 1 < n_kv) issue_s(j + 1);
        issue_pv(j);
      }
      if (ok && ptx::elect_one()) ptx::tc_commit(o_done);
    }
  } else {
    const int q = warp & 3;                            // TMEM lane quadrant
    const int r = q * 32 + lane;                       // query row inside the tile
    const int qi = qt * BQ + r;                        // position
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    float m_used = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv && ok; ++j) {
      const int sb = j & 1;
      ok = ptx::mbar_wait(&s_full[sb], (j >> 1) & 1, abort_flag, g.status);
      if (!ok) break;
      ptx::tc_fence_after();
      const uint32_t ts = tmem_base + TM_S + sb * BKV + lane_addr;
      const bool diag = (j >= 2 * qt);                 // the two 64-key blocks that straddle this tile's diagonal
      const int kj0 = j * BKV;
      // the whole score row of this thread: four loads in flight, one wait
      uint32_t rv[BKV];
#pragma unroll
      for (int ch = 0; ch < BKV / 32; ++ch) ptx::tmem_ld32(ts + ch * 32, rv + ch * 32);
      ptx::tmem_ld_wait();
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // row maximum (log2 domain), four independent chains
      if (diag) {
#pragma unroll
        for (int c = 0; c < BKV; ++c)
          if (kj0 + c <= qi) mx4[c & 3] = fmaxf(mx4[c & 3], __uint_as_float(rv[c]));
      } else {
#pragma unroll
        for (int c = 0; c < BKV; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], __uint_as_float(rv[c]));
      }
      float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * g.scale_log2;   // the scale is positive
      float corr = 1.f;
      bool rescale = false;
      if (mx > m_used + kRescaleThreshold) {           // (first tile: m_used = -inf)
        corr = ex2(m_used - mx);                       // 0 on the first tile
        l *= corr;
        m_used = mx;
        rescale = j > 0;
      }
      // p = 2^(s - m), packed to bf16 for the second MMA
      uint32_t pk[BKV / 2];
      float l0 = 0.f, l1 = 0.f;
#pragma unroll
      for (int c = 0; c < BKV; c += 2) {
        float p0 = ex2(fmaf(__uint_as_float(rv[c]), g.scale_log2, -m_used));
        float p1 = ex2(fmaf(__uint_as_float(rv[c + 1]), g.scale_log2, -m_used));
        if (diag) {
          if (kj0 + c > qi) p0 = 0.f;
          if (kj0 + c + 1 > qi) p1 = 0.f;
        }
        l0 += p0;
        l1 += p1;
        pk[c / 2] = float2_to_bf16x2(p0, p1);
      }
      l += l0 + l1;
      if (__any_sync(0xFFFFFFFFu, rescale)) {
        // O is rescaled in place: the previous P V, which accumulates into it, must have completed
        ok = ptx::mbar_wait(p_empty, (j & 1) ^ 1, abort_flag, g.status);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t to = tmem_base + TM_O + lane_addr;
#pragma unroll 1
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t ro[32];
          ptx::tmem_ld32(to + ch * 32, ro);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 32; ++c) ro[c] = __float_as_uint(__uint_as_float(ro[c]) * (rescale ? corr : 1.f));
          ptx::tmem_st32(to + ch * 32, ro);
        }
        ptx::tmem_st_wait();
      }
      // P row r (bf16 pairs) over the first 32 columns of the S buffer this thread has just read: each
      // warp touches only its own lanes, and the buffer is not reused before P V (j) has completed
      ptx::tmem_st32(ts, pk);
      ptx::tmem_st_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(p_full);
    }
    if (ok) ok = ptx::mbar_wait(o_done, 0, abort_flag, g.status);
    if (ok) {
      ptx::tc_fence_after();
      const float inv = 1.f / l;
      const bool wide_store = (reinterpret_cast<uintptr_t>(g.out) & 31) == 0 && g.o_sn % 16 == 0 && g.o_sh % 16 == 0 && g.o_st % 16 == 0;
      __nv_bfloat16* orow = g.out + (long long)b * g.o_sn + (long long)h * g.o_sh + (long long)qi * g.o_st;
      const uint32_t to = tmem_base + TM_O + lane_addr;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t rv[32];
        ptx::tmem_ld32(to + ch * 32, rv);
        ptx::tmem_ld_wait();
        if (qi < g.S && wide_store) {                    // whole 32-byte sectors per store
#pragma unroll
          for (int v = 0; v < 2; ++v) {
            uint32_t w[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
              w[e] = float2_to_bf16x2(__uint_as_float(rv[v * 16 + 2 * e]) * inv, __uint_as_float(rv[v * 16 + 2 * e + 1]) * inv);
            ptx::st_global_v8(orow + ch * 32 + v * 16, make_uint4(w[0], w[1], w[2], w[3]), make_uint4(w[4], w[5], w[6], w[7]));
          }
        } else if (qi < g.S) {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            float o8[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) o8[e] = __uint_as_float(rv[v * 8 + e]) * inv;
            ElemIO<__nv_bfloat16>::store(orow + ch * 32 + v * 8, o8);
          }
        }
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

// Returns SMARTMEM_ERR_UNSUPPORTED when the operand layout is neither of the two it knows.
int launch_causal_attention_tc(const CausalAttnArgs& a, cudaStream_t st) {
  const long long S = a.S, H = a.heads, B = a.batch;
  if (S < 1 || H < 1 || B < 1) return SMARTMEM_ERR_UNSUPPORTED;
  const AttnOperand* ops[3] = {&a.q, &a.k, &a.v};
  for (auto* o : ops)
    if (o->se != 1 || ((uintptr_t)o->ptr & 15)) return SMARTMEM_ERR_UNSUPPORTED;
  if (a.o.se != 1 || a.o.st % 8 || a.o.sn % 8 || a.o.sh % 8 || ((uintptr_t)a.o.ptr & 15)) return SMARTMEM_ERR_UNSUPPORTED;
  TcAttnArgs g;
  memset(&g, 0, sizeof(g));
  CUtensorMap tq, tk, tv;
  int rc;
  const long long st_ = a.q.st;
  const bool interleaved = a.q.sh == D && a.k.sh == D && a.v.sh == D && a.k.st == st_ && a.v.st == st_ &&
                           a.q.sn == S * st_ && a.k.sn == S * st_ && a.v.sn == S * st_ && st_ % 8 == 0;
  const bool head_major = a.q.st == D && a.k.st == D && a.v.st == D && a.q.sh == S * D && a.k.sh == S * D &&
                          a.v.sh == S * D && a.q.sn == H * S * D && a.k.sn == H * S * D && a.v.sn == H * S * D;
  if (interleaved) {
    // one [B*S, row pitch] matrix holds q, k and v side by side; columns are offsets from q
    const long long kcol = ((const char*)a.k.ptr - (const char*)a.q.ptr) / 2, vcol = ((const char*)a.v.ptr - (const char*)a.q.ptr) / 2;
    if (kcol < 0 || vcol < 0 || kcol + H * D > st_ || vcol + H * D > st_) return SMARTMEM_ERR_UNSUPPORTED;
    if ((rc = tc_encode_2d(a.q.ptr, st_, B * S, st_, 64, BQ, &tq)) != SMARTMEM_OK) return rc;
    if ((rc = tc_encode_2d(a.q.ptr, st_, B * S, st_, 64, BKV, &tk)) != SMARTMEM_OK) return rc;   // same buffer, 64-row boxes
    tv = tk;
    g.q_col0 = 0; g.k_col0 = (int)kcol; g.v_col0 = (int)vcol; g.col_per_head = D;
    g.row_per_batch = S; g.row_per_head = 0;
  } else if (head_major) {
    if ((rc = tc_encode_2d(a.q.ptr, D, B * H * S, D, 64, 128, &tq)) != SMARTMEM_OK) return rc;
    if ((rc = tc_encode_2d(a.k.ptr, D, B * H * S, D, 64, BKV, &tk)) != SMARTMEM_OK) return rc;
    if ((rc = tc_encode_2d(a.v.ptr, D, B * H * S, D, 64, BKV, &tv)) != SMARTMEM_OK) return rc;
    g.col_per_head = 0;
    g.row_per_batch = H * S; g.row_per_head = S;
  } else {
    return SMARTMEM_ERR_UNSUPPORTED;
  }
  if (B * H * S >= (1ll << 31)) return SMARTMEM_ERR_UNSUPPORTED;
  g.S = (int)S; g.heads = (int)H; g.batch = (int)B;
  g.n_qt = (int)((S + BQ - 1) / BQ);
  g.out = (__nv_bfloat16*)a.o.ptr;
  g.o_sn = a.o.sn; g.o_sh = a.o.sh; g.o_st = a.o.st;
  g.scale_log2 = a.scale * 1.4426950408889634f;
  g.status = device_status_ptr();
  if (!g.status) return SMARTMEM_ERR_CUDA;
  // 112 KB of tiles: two CTAs per SM only fit without a spare kilobyte of alignment slack (the kernel
  // reports a misaligned base instead of overrunning)
  const size_t smem = 2 * KB + 8 * KBK + 16 * 8 + 16;
  g.smem_bytes = (uint32_t)smem;
  if (ensure_max_dynamic_smem((const void*)causal_attn_tc_kernel, (int)smem, 100) != SMARTMEM_OK) return SMARTMEM_ERR_CUDA;
  const long long ctas = (long long)g.n_qt * B * H;
  if (ctas >= (1ll << 31)) return SMARTMEM_ERR_UNSUPPORTED;
  profile_tick("causal_attention_tc", st);
  launch_pdl(causal_attn_tc_kernel, dim3((unsigned)ctas), dim3(kThreads), smem, st, tq, tk, tv, g);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

}  // namespace smartmem
