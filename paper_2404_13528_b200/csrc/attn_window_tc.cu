// Window attention (head dimension 32, T = ws*ws <= 64) on the tcgen05 tensor cores.
//
// Two windows of one head share a 128-row MMA tile: S = [Q0; Q1] [K0; K1]^T is computed as one
// 128 x 128 x 32 product (only its two diagonal 64 x 64 blocks are used) and O = P [V0; V1] as one
// 128 x 32 x 128 product with a block-diagonal P, so each window only sees its own keys.  The tensor
// core has time to spare here; what the layout buys is that every query row belongs to exactly one
// thread (its TMEM lane): bias, mask, maximum, exponentials and the row sum need no shuffles, no
// fragment bookkeeping and no shared-memory fragment loads, which is what bounded the warp-MMA
// version (it was instruction-issue bound).
//
// q, k, v are TMA boxes of 64 rows x 32 columns inside the [M, 3C] buffer of the QKV GEMM (head
// split, K transpose eliminated); operands that TMA cannot address (the materialised K^T of the
// explicit variant) are loaded by four helper warps into the same swizzled layout.  V is used as it
// lies ([key, d] rows) through the MN-major operand mode.  Results are stored as whole 64-byte rows
// at column h*32 of [M, C] (head merge eliminated) or into [nW, nH, T, d].
//
// Persistent CTAs keep one head (its relative-position bias is expanded once into a [T, T] table of
// bf16 pairs in shared memory, read with 16-byte loads) and stream window pairs through a 6-stage
// ring.  Two softmax groups of four warps alternate over the units, each with its own S and O buffers
// and its own P region in TMEM (P is written there as bf16 pairs and read by the second MMA as its
// A operand: it never touches shared memory).  S and P V have an issuing thread each: the S issuer runs ahead as far
// as the S buffers and the ring allow, so a group finds its next score tile waiting when it has
// written P.  The seam mask of shifted blocks is a 64-bit key mask per row, computed arithmetically
// (a key is in another region iff it lies on the other side of the wrap line) and only for windows
// in the last window row or column.
//
// What bounds it (measured with clock stamps at every hand-off): the softmax groups, at about 1700 cycles
// per window pair; the tensor pipe is busy for about 500 of them.
#include "attn.cuh"
#include "gemm_tc.cuh"
#include "ptx.cuh"


namespace smartmem {
namespace {

constexpr int D = 32, TP = 64;
constexpr int OP_BYTES = 128 * 64;                    // one operand of a pair: 128 rows x 64 bytes
constexpr int STAGE_BYTES = 3 * OP_BYTES;             // q, k, v
constexpr int NSTAGE = 6;
constexpr uint32_t TM_S = 0, TM_O = 256, TM_P = 320, TMEM_COLS = 512;   // S 2 x 128 columns, O 2 x 32, P 2 x 64 (128 keys as bf16 pairs)
constexpr int BIAS_ROW = 36;                          // 32-bit words per bias row: 64 bf16 + pad, so that 16-byte row reads of
                                                      // eight consecutive threads fall into distinct banks
constexpr int kSoftmaxWarps = 4, kGroups = 2, kLoaderWarps = 4;   // two softmax groups alternate over the units
constexpr int kThreads = 32 * (3 + kGroups * kSoftmaxWarps + kLoaderWarps);   // + producer, P V issuer, S issuer

struct WinTcArgs {
  WinAttnArgs a;
  int n_pairs, tma_mask;                               // bit m set: operand m (q, k, v) comes through TMA
  FastDiv fd_T;
  int col0[3], col_per_head[3];                        // TMA column of (operand, head)
  long long row_per_window[3], row_per_head[3];        // TMA row of (window, head): n * rpw + h * rph
  int* status;
};

// Shared-memory matrix descriptor with 64-byte swizzle (rows of 64 bytes, 8-row groups 512 bytes apart).
__device__ __forceinline__ uint64_t make_desc_sw64(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)4 << 61;
  return d;
}

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// KC: key columns a softmax thread works on (56 when the window has at most 56 tokens -- a 7 x 7 window
// has 49 -- else 64).  Columns [T, 64) of a score row are padding whose probability is zero.
template <int KC>
__global__ void __launch_bounds__(kThreads, 1)
win_attn_tc_kernel(const __grid_constant__ CUtensorMap tm0, const __grid_constant__ CUtensorMap tm1,
                   const __grid_constant__ CUtensorMap tm2, const __grid_constant__ WinTcArgs g) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  uint8_t* sIn = smem;                                 // [NSTAGE][q, k, v][128 rows x 64 B]
  uint32_t* bias_s = reinterpret_cast<uint32_t*>(sIn + NSTAGE * STAGE_BYTES);   // [64][36]: bf16 pairs, 144-byte rows
  int* lab_s = reinterpret_cast<int*>(bias_s + TP * BIAS_ROW);   // scratch: the head's raw table column (<= 256 bf16), then 4 key-mask words
  uint16_t* raw_s = reinterpret_cast<uint16_t*>(lab_s);
  uint32_t* kmask_s = reinterpret_cast<uint32_t*>(lab_s) + 128;
  int* tyx_s = lab_s + kGroups * 2 * TP;                         // [64]: ty << 8 | tx
  uint64_t* bars = reinterpret_cast<uint64_t*>(tyx_s + TP);
  uint64_t *in_full = bars, *in_empty = bars + NSTAGE, *s_full = bars + 2 * NSTAGE, *s_empty = s_full + 2;
  uint64_t *p_full = s_empty + 2, *p_empty = p_full + 2, *o_full = p_empty + 2, *o_empty = o_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_empty + 2);
  int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);

  const WinAttnArgs& a = g.a;
  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0);   // (provably warp-uniform: the issuer warps keep their operands in uniform registers)
  const int T = a.T, ws = a.ws;
  const int h = blockIdx.x % a.heads;
  const int cidx = blockIdx.x / a.heads, cstride = gridDim.x / a.heads;
  const bool any_manual = g.tma_mask != 7;
  const float LOG2E = 1.4426950408889634f;

  if (tid == 0) {
    for (int i = 0; i < NSTAGE; ++i) {
      ptx::mbar_init(&in_full[i], 1 + (any_manual ? 32 * kLoaderWarps : 0));
      ptx::mbar_init(&in_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&s_full[i], 1);
      ptx::mbar_init(&s_empty[i], kSoftmaxWarps);
      ptx::mbar_init(&o_full[i], 1);
      ptx::mbar_init(&o_empty[i], kSoftmaxWarps);
    }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&p_full[i], kSoftmaxWarps);
      ptx::mbar_init(&p_empty[i], 1);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (warp == 1) ptx::tmem_alloc(tmem_slot, TMEM_COLS);   // first: its latency overlaps the table set-up below
  // one-time tables.  First the inputs of the table (one global load per thread, one latency): the
  // head's column of the relative-position table and the token coordinates; P's off-diagonal blocks
  // (and, for hand-loaded operands, the padded rows of the input stages) are zeroed meanwhile.
  const int n_table = (2 * ws - 1) * (2 * ws - 1);
  for (int i = tid; i < n_table && i < 256; i += kThreads) raw_s[i] = reinterpret_cast<const uint16_t*>(a.table)[i * a.heads + h];
  if (tid < TP) tyx_s[tid] = ((tid / ws) << 8) | (tid % ws);
  {
    uint8_t* z0 = smem;
    const int zbytes = any_manual ? NSTAGE * STAGE_BYTES : 0;
    for (int i = tid; i < zbytes / 16; i += kThreads) reinterpret_cast<uint4*>(z0)[i] = make_uint4(0, 0, 0, 0);
  }
  __syncthreads();
  // the head's bias as a [T, T] table of bf16 pairs, -inf for padded keys
  for (int i = tid; i < TP * (TP / 2); i += kThreads) {
    const int r = i / (TP / 2), c2 = i - r * (TP / 2);
    const int ry = tyx_s[r] >> 8, rx = tyx_s[r] & 255;
    uint32_t word = 0;
    for (int k = 0; k < 2; ++k) {
      const int c = 2 * c2 + k;
      uint32_t bits = 0;                               // bf16 bit pattern
      if (c >= T) {
        bits = 0xFF80u;                                // -inf: padded keys never contribute
      } else if (r < T) {
        const int cy = tyx_s[c] >> 8, cx = tyx_s[c] & 255;
        bits = raw_s[(ry - cy + ws - 1) * (2 * ws - 1) + (rx - cx + ws - 1)];
      }
      word |= bits << (16 * k);
    }
    bias_s[r * BIAS_ROW + c2] = word;
  }
  // keys below / right of the wrap line of a seam window (bit c = key c)
  if (warp == 2) {
    const int c0 = lane, c1 = lane + 32;
    const bool y0 = c0 < T && (tyx_s[c0] >> 8) >= ws - a.shift, y1 = c1 < T && (tyx_s[c1] >> 8) >= ws - a.shift;
    const bool x0 = c0 < T && (tyx_s[c0] & 255) >= ws - a.shift, x1 = c1 < T && (tyx_s[c1] & 255) >= ws - a.shift;
    const uint32_t m0 = __ballot_sync(0xFFFFFFFFu, y0), m1 = __ballot_sync(0xFFFFFFFFu, y1);
    const uint32_t m2 = __ballot_sync(0xFFFFFFFFu, x0), m3 = __ballot_sync(0xFFFFFFFFu, x1);
    if (lane == 0) { kmask_s[0] = m0; kmask_s[1] = m1; kmask_s[2] = m2; kmask_s[3] = m3; }
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(&tm0);
    ptx::prefetch_tensormap(&tm1);
    ptx::prefetch_tensormap(&tm2);
  }
  ptx::fence_proxy_async();
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                       // the tables above depend on parameters only: they overlapped the previous kernel's tail
  pdl_launch_dependents();
  const CUtensorMap* tms[3] = {&tm0, &tm1, &tm2};
  const AttnOperand* ops[3] = {&a.q, &a.k, &a.v};

  if (warp == 0) {
    // ---- TMA producer ------------------------------------------------------------------------
    if (lane == 0) {
      int n_tma = 0;
      for (int m = 0; m < 3; ++m) n_tma += (g.tma_mask >> m) & 1;
      bool ok = true;
      uint32_t it = 0;
      for (int p = cidx; p < g.n_pairs && ok; p += cstride, ++it) {
        const int s = it % NSTAGE;
        ok = ptx::mbar_wait(&in_empty[s], ((it / NSTAGE) & 1) ^ 1, abort_flag, g.status);
        if (!ok) break;
        const int nwin = (2 * p + 1 < a.n_windows) ? 2 : 1;
        ptx::mbar_expect_tx(&in_full[s], (uint32_t)(n_tma * nwin * TP * 64));
        for (int m = 0; m < 3; ++m) {
          if (!((g.tma_mask >> m) & 1)) continue;
          for (int w = 0; w < nwin; ++w) {
            const long long n = 2 * p + w;
            ptx::tma_load_2d(sIn + s * STAGE_BYTES + m * OP_BYTES + w * (TP * 64), tms[m], &in_full[s],
                             g.col0[m] + h * g.col_per_head[m], (int)(n * g.row_per_window[m] + h * g.row_per_head[m]));
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---- P V issuer (and owner of the tensor memory): the whole warp walks the loop, an elected lane issues ----
    {
      const uint32_t idesc_pv = ptx::make_idesc_bf16(128, D, false, true);     // V: MN-major B operand
      bool ok = true;
      const int my_units = cidx < g.n_pairs ? (g.n_pairs - cidx + cstride - 1) / cstride : 0;
      for (int u = 0; u < my_units && ok; ++u) {
        const int s = u % NSTAGE, ob = u & 1;
        ok = ptx::mbar_wait(&p_full[ob], (u >> 1) & 1, abort_flag, g.status);
        ok = ok && ptx::mbar_wait(&o_empty[ob], ((u >> 1) & 1) ^ 1, abort_flag, g.status);
        ok = __all_sync(0xFFFFFFFFu, ok ? 1 : 0) != 0;
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t v0 = ptx::smem_u32(sIn + s * STAGE_BYTES + 2 * OP_BYTES);
        const uint64_t vd = make_desc_sw64(v0, 16, 512);
        const uint32_t od = tmem_base + TM_O + ob * D, pa = tmem_base + TM_P + ob * 64;
        if (ptx::elect_one()) {
          ptx::tc_mma_bf16_ta(od, pa, vd, idesc_pv, 0u);
#pragma unroll
          for (int ks = 1; ks < 8; ++ks)               // 16 keys per step: P +8 packed columns, V +1024 bytes
            ptx::tc_mma_bf16_ta(od, pa + 8 * ks, vd + ks * (1024 >> 4), idesc_pv, 1u);
          ptx::tc_commit(&in_empty[s]);
          ptx::tc_commit(&p_empty[ob]);
          ptx::tc_commit(&o_full[ob]);
        }
        __syncwarp();
      }
    }
  } else if (warp == 2 + kGroups * kSoftmaxWarps + kLoaderWarps) {
    // ---- S issuer: runs ahead of P V as far as the two S buffers and the input ring allow, so a
    // softmax group finds its next score tile waiting when it has written P ---------------------
    {
      const uint32_t idesc_s = ptx::make_idesc_bf16(128, 128, false, false);
      bool ok = true;
      const int my_units = cidx < g.n_pairs ? (g.n_pairs - cidx + cstride - 1) / cstride : 0;
      for (int u = 0; u < my_units && ok; ++u) {
        const int s = u % NSTAGE, sb = u & 1;
        ok = ptx::mbar_wait(&s_empty[sb], ((u >> 1) & 1) ^ 1, abort_flag, g.status);
        ok = ok && ptx::mbar_wait(&in_full[s], (u / NSTAGE) & 1, abort_flag, g.status);
        ok = __all_sync(0xFFFFFFFFu, ok ? 1 : 0) != 0;
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t q0 = ptx::smem_u32(sIn + s * STAGE_BYTES), k0 = q0 + OP_BYTES;
        const uint64_t qd = make_desc_sw64(q0, 16, 512), kd = make_desc_sw64(k0, 16, 512);
        if (ptx::elect_one()) {
          ptx::tc_mma_bf16(tmem_base + TM_S + sb * 128, qd, kd, idesc_s, 0u);
          ptx::tc_mma_bf16(tmem_base + TM_S + sb * 128, qd + 2, kd + 2, idesc_s, 1u);  // next 16 features: +32 bytes
          ptx::tc_commit(&s_full[sb]);
        }
        __syncwarp();
      }
    }
  } else if (warp < 2 + kGroups * kSoftmaxWarps) {
    // ---- softmax + epilogue: one query row per thread; group gi takes the units u = gi (mod 2) ----
    const int gi = (warp - 2) / kSoftmaxWarps;
    const int q = warp & 3;                            // TMEM lane quadrant
    const int r = q * 32 + lane;                       // row of the pair tile
    const int w = r >> 6, i = r & 63;                  // window of the pair, token
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    const int my_ty = tyx_s[i] >> 8, my_tx = tyx_s[i] & 255;
    const uint32_t* brow = bias_s + i * BIAS_ROW;
    {                                                  // block-diagonal P: the other window's keys contribute nothing to this row
      uint32_t zero[32];
#pragma unroll
      for (int c = 0; c < 32; ++c) zero[c] = 0u;
      ptx::tmem_st32(tmem_base + TM_P + gi * 64 + lane_addr + (1 - w) * 32, zero);
      ptx::tmem_st_wait();
    }
    // keys below / right of the wrap line of a seam window (bit c = key c), and this row's own side
    const uint32_t ky_lo = kmask_s[0], ky_hi = kmask_s[1], kx_lo = kmask_s[2], kx_hi = kmask_s[3];
    const uint32_t my_fy = my_ty >= ws - a.shift ? 0xFFFFFFFFu : 0u, my_fx = my_tx >= ws - a.shift ? 0xFFFFFFFFu : 0u;
    float inv_prev = 0.f;
    int n_prev = -1;
    bool ok = true;
    const bool wide_store = (reinterpret_cast<uintptr_t>(a.o.ptr) & 31) == 0 && a.o.sn % 16 == 0 && a.o.sh % 16 == 0 && a.o.st % 16 == 0;
    auto epilogue = [&](int u, float inv, int n) {     // O(u) -> global
      const int ob = u & 1;                            // == gi
      ok = ok && ptx::mbar_wait(&o_full[ob], (u >> 1) & 1, abort_flag, g.status);
      if (!ok) return;
      ptx::tc_fence_after();
      uint32_t rv[32];
      ptx::tmem_ld32(tmem_base + TM_O + ob * D + lane_addr, rv);
      ptx::tmem_ld_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&o_empty[ob]);
      if (i < T && n < a.n_windows) {
        __nv_bfloat16* dst = (__nv_bfloat16*)a.o.ptr + (long long)n * a.o.sn + (long long)h * a.o.sh + (long long)i * a.o.st;
        if (wide_store) {                              // whole 32-byte sectors per store
#pragma unroll
          for (int v = 0; v < 2; ++v) {
            uint32_t w[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
              w[e] = float2_to_bf16x2(__uint_as_float(rv[v * 16 + 2 * e]) * inv, __uint_as_float(rv[v * 16 + 2 * e + 1]) * inv);
            ptx::st_global_v8(dst + v * 16, make_uint4(w[0], w[1], w[2], w[3]), make_uint4(w[4], w[5], w[6], w[7]));
          }
        } else {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            float o8[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) o8[e] = __uint_as_float(rv[v * 8 + e]) * inv;
            ElemIO<__nv_bfloat16>::store(dst + v * 8, o8);
          }
        }
      }
    };
    int u = gi;
    int done = 0;
    for (int p = cidx + gi * cstride; p < g.n_pairs && ok; p += 2 * cstride, u += 2, ++done) {
      const int sb = u & 1;
      const int n = 2 * p + w;
      // Shifted blocks: only windows in the last window row or column straddle the seam.  There a key
      // lies in another region than this row iff the two sit on different sides of the wrap line at
      // ws - shift, vertically (last window row) or horizontally (last window column): one 64-bit
      // mask per row, from the two key masks computed once above.
      bool masked = false;
      uint32_t diff_lo = 0, diff_hi = 0;
      if (a.shift > 0 && n < a.n_windows) {
        const int wl = n - (int)fd_div((uint32_t)n, a.fd_wpi) * a.win_per_img;
        const int wy = (int)fd_div((uint32_t)wl, a.fd_nww), wx = wl - wy * a.nWw;
        const bool last_row = wy == a.nWh - 1, last_col = wx == a.nWw - 1;
        masked = last_row || last_col;
        if (last_row) { diff_lo |= ky_lo ^ my_fy; diff_hi |= ky_hi ^ my_fy; }
        if (last_col) { diff_lo |= kx_lo ^ my_fx; diff_hi |= kx_hi ^ my_fx; }
      }
      ok = ptx::mbar_wait(&s_full[sb], (u >> 1) & 1, abort_flag, g.status);
      if (!ok) break;
      ptx::tc_fence_after();
      uint32_t rv[KC];
      const uint32_t ts = tmem_base + TM_S + sb * 128 + lane_addr + w * 64;    // this window's 64 key columns
      ptx::tmem_ld32(ts, rv);
      if constexpr (KC == 64) {
        ptx::tmem_ld32(ts + 32, rv + 32);
      } else {
        ptx::tmem_ld16(ts + 32, rv + 32);
        ptx::tmem_ld8(ts + 48, rv + 48);
      }
      ptx::tmem_ld_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&s_empty[sb]);
      float sc[KC];
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // independent chains
      // scores in natural units: q.k * scale + bias (the row's 64 biases come as eight 16-byte reads
      // of bf16 pairs); the base-2 conversion is folded into the exponent's multiply-add below
#pragma unroll
      for (int v8 = 0; v8 < KC / 8; ++v8) {
        const uint4 b4 = *reinterpret_cast<const uint4*>(brow + v8 * 4);
        const uint32_t bw[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int c = v8 * 8 + 2 * j;
          sc[c] = fmaf(__uint_as_float(rv[c]), a.scale, __uint_as_float(bw[j] << 16));
          sc[c + 1] = fmaf(__uint_as_float(rv[c + 1]), a.scale, __uint_as_float(bw[j] & 0xFFFF0000u));
        }
      }
      if (masked) {                                    // seam windows only: keys of another region get -100
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
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t pk[32];
#pragma unroll
      for (int c = KC / 2; c < 32; ++c) pk[c] = 0u;        // padding keys
#pragma unroll
      for (int c = 0; c < KC; c += 2) {
        const float p0 = ex2f(fmaf(sc[c], LOG2E, nmx)), p1 = ex2f(fmaf(sc[c + 1], LOG2E, nmx));
        sum4[c & 2] += p0;
        sum4[(c & 2) + 1] += p1;
        pk[c / 2] = float2_to_bf16x2(p0, p1);
      }
      const float inv = 1.f / ((sum4[0] + sum4[1]) + (sum4[2] + sum4[3]));
      // drain this group's previous unit: its P V has finished by now, and the O buffer it frees is
      // the one this unit's P V accumulates into
      if (done > 0) epilogue(u - 2, inv_prev, n_prev);
      if (!ok) break;
      // previous P V must have completed before P is overwritten
      ok = ptx::mbar_wait(&p_empty[gi], ((u >> 1) & 1) ^ 1, abort_flag, g.status);
      if (!ok) break;
      // P row r (bf16 pairs): its window's 64 keys are packed columns w*32 .. w*32+31 of the group's P region;
      // the other window's half of the row was zeroed once and is never written
      ptx::tc_fence_after();
      ptx::tmem_st32(tmem_base + TM_P + gi * 64 + lane_addr + w * 32, pk);
      ptx::tmem_st_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&p_full[gi]);
      inv_prev = inv;
      n_prev = n;
    }
    if (ok && done > 0) epilogue(u - 2, inv_prev, n_prev);
  } else if (warp < 2 + kGroups * kSoftmaxWarps + kLoaderWarps) {
    // ---- helper loaders for operands TMA cannot address (e.g. a materialised K^T) ----------------
    if (any_manual) {
      const int lt = tid - 32 * (2 + kGroups * kSoftmaxWarps);
      bool ok = true;
      uint32_t it = 0;
      for (int p = cidx; p < g.n_pairs && ok; p += cstride, ++it) {
        const int s = it % NSTAGE;
        ok = ptx::mbar_wait(&in_empty[s], ((it / NSTAGE) & 1) ^ 1, abort_flag, g.status);
        if (!ok) break;
        for (int m = 0; m < 3; ++m) {
          if ((g.tma_mask >> m) & 1) continue;
          const AttnOperand& o = *ops[m];
          uint8_t* dst = sIn + s * STAGE_BYTES + m * OP_BYTES;
          // A window's operand is one contiguous block of T*D elements when it is a materialised
          // [T, d] or [d, T] matrix: read it with 16-byte loads and scatter the 8 elements of a load
          // to their (token, feature) slots of the swizzled tile.
          const bool block_td = o.se == 1 && o.st == D, block_dt = o.st == 1 && o.se == T;
          const bool vec_ok = (block_td || block_dt) && (T * D) % 8 == 0 && o.sn % 8 == 0 && o.sh % 8 == 0 &&
                              ((uintptr_t)o.ptr & 15) == 0;
          auto put = [&](int w, int t, int e, __nv_bfloat16 v) {
            const int row = w * TP + t;                // 64-byte rows, 16-byte chunks swizzled by (row / 2) % 4
            *reinterpret_cast<__nv_bfloat16*>(dst + row * 64 + ((((e >> 3) ^ ((row >> 1) & 3))) << 4) + (e & 7) * 2) = v;
          };
          if (vec_ok) {
            const int nvec = T * D / 8;
            for (int idx = lt; idx < 2 * nvec; idx += 32 * kLoaderWarps) {
              const int w = idx >= nvec ? 1 : 0, vi = idx - w * nvec;
              const long long n = 2 * p + w;
              uint4 raw = make_uint4(0, 0, 0, 0);
              if (n < a.n_windows)
                raw = *reinterpret_cast<const uint4*>((const __nv_bfloat16*)o.ptr + n * o.sn + (long long)h * o.sh + vi * 8);
              const __nv_bfloat16* ev = reinterpret_cast<const __nv_bfloat16*>(&raw);
              // (token, feature) of the first element: one reciprocal division, then counting
              int t, e;
              if (block_td) { t = (vi * 8) >> 5; e = (vi * 8) & 31; }
              else { e = (int)fd_div((uint32_t)(vi * 8), g.fd_T); t = vi * 8 - e * T; }
#pragma unroll
              for (int k = 0; k < 8; ++k) {
                put(w, t, e, ev[k]);
                if (block_td) { if (++e == D) { e = 0; ++t; } }
                else { if (++t == T) { t = 0; ++e; } }
              }
            }
          } else {
            for (int idx = lt; idx < 2 * T * D; idx += 32 * kLoaderWarps) {
              const int w = idx / (T * D), rem = idx - w * (T * D);
              int t, e;
              if (o.se == 1) { t = rem / D; e = rem - t * D; } else { e = rem / T; t = rem - e * T; }
              const long long n = 2 * p + w;
              __nv_bfloat16 v = __float2bfloat16_rn(0.f);
              if (n < a.n_windows)
                v = ((const __nv_bfloat16*)o.ptr)[n * o.sn + (long long)h * o.sh + (long long)t * o.st + (long long)e * o.se];
              put(w, t, e, v);
            }
          }
        }
        ptx::fence_proxy_async();
        ptx::mbar_arrive(&in_full[s]);
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

// Returns SMARTMEM_ERR_UNSUPPORTED for shapes the kernel does not cover (the caller then uses the
// warp-MMA kernel).
int launch_window_attention_tc(const WinAttnArgs& a_in, long long n_windows, cudaStream_t st) {
  if (a_in.table_f32) return SMARTMEM_ERR_UNSUPPORTED;     // the bias table is kept as bf16 pairs
  if (a_in.d != D || a_in.T > TP || a_in.T < 1 || n_windows < 1 || n_windows >= (1ll << 30)) return SMARTMEM_ERR_UNSUPPORTED;
  if (a_in.o.se != 1 || a_in.o.st % 8 || a_in.o.sn % 8 || a_in.o.sh % 8 || ((uintptr_t)a_in.o.ptr & 15)) return SMARTMEM_ERR_UNSUPPORTED;
  WinTcArgs g;
  memset(&g, 0, sizeof(g));
  g.a = a_in;
  WinAttnArgs& a = g.a;
  a.n_windows = (int)n_windows;
  a.nWh = a.win_per_img / a.nWw;
  a.fd_wpi = make_fastdiv((uint32_t)a.win_per_img);
  a.fd_nww = make_fastdiv((uint32_t)a.nWw);
  g.n_pairs = (int)((n_windows + 1) / 2);
  g.fd_T = make_fastdiv((uint32_t)a.T);
  g.status = device_status_ptr();
  if (!g.status) return SMARTMEM_ERR_CUDA;
  CUtensorMap tm[3];
  memset(tm, 0, sizeof(tm));
  const AttnOperand* ops[3] = {&a.q, &a.k, &a.v};
  const long long T = a.T, H = a.heads;
  for (int m = 0; m < 3; ++m) {
    const AttnOperand& o = *ops[m];
    // rows of 32 contiguous elements, 16-byte aligned pitch; two addressing patterns
    const bool rows_ok = o.se == 1 && o.st % 8 == 0 && ((uintptr_t)o.ptr & 15) == 0;
    if (rows_ok && o.sh == D && o.sn == T * o.st) {                 // [M, pitch] with heads side by side
      if (tc_encode_2d_sw64(o.ptr, H * D, n_windows * T, o.st, D, TP, &tm[m]) != SMARTMEM_OK) continue;
      g.col0[m] = 0; g.col_per_head[m] = D; g.row_per_window[m] = T; g.row_per_head[m] = 0;
      g.tma_mask |= 1 << m;
    } else if (rows_ok && o.st == D && o.sh == T * D && o.sn == H * T * D) {     // [nW, nH, T, d]
      if (tc_encode_2d_sw64(o.ptr, D, n_windows * H * T, D, D, TP, &tm[m]) != SMARTMEM_OK) continue;
      g.col0[m] = 0; g.col_per_head[m] = 0; g.row_per_window[m] = H * T; g.row_per_head[m] = T;
      g.tma_mask |= 1 << m;
    }
  }
  const size_t smem = 1024 + NSTAGE * STAGE_BYTES + TP * BIAS_ROW * 4 + (2 * kGroups + 1) * TP * 4 +
                      (2 * NSTAGE + 12) * 8 + 16;
  if (ensure_max_dynamic_smem((const void*)win_attn_tc_kernel<56>, (int)smem) != SMARTMEM_OK ||
      ensure_max_dynamic_smem((const void*)win_attn_tc_kernel<64>, (int)smem) != SMARTMEM_OK)
    return SMARTMEM_ERR_CUDA;
  const int sms = tc_sm_count();
  long long per_head = (long long)sms / a.heads;
  if (per_head < 1) per_head = 1;
  if (per_head > g.n_pairs) per_head = g.n_pairs;
  const unsigned grid = (unsigned)(per_head * a.heads);
  profile_tick("window_attention_tc", st);
  if (a.T <= 56) launch_pdl(win_attn_tc_kernel<56>, dim3(grid), dim3(kThreads), smem, st, tm[0], tm[1], tm[2], g);
  else launch_pdl(win_attn_tc_kernel<64>, dim3(grid), dim3(kThreads), smem, st, tm[0], tm[1], tm[2], g);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

}  // namespace smartmem
