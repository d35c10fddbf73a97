// Window attention: softmax(d^-1/2 q k^T + relative-position bias [+ shifted-window mask]) v
// for one (window, head) per CTA.
//
// The head split (Reshape -> Transpose -> Slice), the K transpose and the head merge
// (Transpose -> Reshape) around it are eliminated: q, k and v are read where the QKV GEMM left
// them (rows of a [M, 3C] buffer, reduction dimension d contiguous for both MMA operands) and
// the result goes straight into the [M, C] layout the projection GEMM reads.  Each operand is
// described by four strides, so the same kernel also consumes the materialised tensors of
// the explicit-layout variant (including a materialised K^T).
//
// Bias and mask are never read from memory as [T,T] tensors: the bias index is
// code(i) - code(j) + const with code(t) = (t div ws)(2ws-1) + t mod ws, looked up in the head's
// column of the table (staged in shared memory); the mask compares per-token region labels
// computed from the window's position.
//
// T = ws*ws <= 64 and d <= 32 make tiles far smaller than a tcgen05 instruction (128 x N), and the
// kernel is bound by HBM traffic (it reads 3 M C and writes M C elements for 4 M T d flops), so the
// contractions use warp-level mma.sync m16n8k16: four warps, 16 query rows each.
#include <cstdlib>

#include "attn.cuh"
#include "ptx.cuh"

namespace smartmem {
namespace {

constexpr int TP = 64;   // padded token count

template <typename T>
__device__ __forceinline__ const T* unit_ptr(const AttnOperand& o, int n, int h) {
  return (const T*)o.ptr + (long long)n * o.sn + (long long)h * o.sh;
}

__device__ __forceinline__ int region_label(int t, int ws, int wy, int wx, int H, int W, int shift) {
  const int hp = wy * ws + t / ws, wp = wx * ws + t % ws;
  const int rh = hp < H - ws ? 0 : (hp < H - shift ? 1 : 2);
  const int rw = wp < W - ws ? 0 : (wp < W - shift ? 1 : 2);
  return 3 * rh + rw;
}

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ptx::smem_u32(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Persistent CTAs (4 warps, one 16-query-row tile each).  A CTA keeps one head: the head's
// relative-position bias for this thread's score fragment is gathered once into registers, and
// the CTA then streams windows through a double-buffered shared-memory pipeline (cp.async), so a
// score element costs one fused multiply-add plus the softmax, and loads overlap the MMAs.
template <int D>
__global__ void __launch_bounds__(128) win_attn_bf16_kernel(const __grid_constant__ WinAttnArgs a) {
  pdl_wait();
  pdl_launch_dependents();
  constexpr int RS = D + 8;                     // padded row (bf16 elements): conflict-free fragment loads
  constexpr int RW = RS / 2;
  constexpr int TILE = TP * RS;
  __shared__ __align__(16) __nv_bfloat16 bufs[2][3][TILE];
  __shared__ int lab_s[2][TP];

  const int T = a.T, ws = a.ws;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
  const int h = blockIdx.x % a.heads;
  const int cidx = blockIdx.x / a.heads, cstride = gridDim.x / a.heads;
  const int r0 = warp * 16 + g, r1 = r0 + 8;
  const bool warp_active = warp * 16 < T;

  // rows >= T of every tile stay zero for the whole kernel
  for (int i = tid; i < 2 * 3 * TILE / 8; i += 128) reinterpret_cast<uint4*>(&bufs[0][0][0])[i] = make_uint4(0, 0, 0, 0);

  // token coordinates: divisions by the (run-time) window size happen once per thread, here
  __shared__ int code_s[TP];
  const int my_ty = tid / ws, my_tx = tid - my_ty * ws;      // token `tid` of a window (tid < 64 used)
  if (tid < TP) code_s[tid] = my_ty * (2 * ws - 1) + my_tx;
  __syncthreads();
  // bias fragment of this head: element (row, col) <- table[(dy + ws - 1)(2ws - 1) + dx + ws - 1, h]
  //                                                 = table[code(row) - code(col) + (ws - 1) 2 ws, h]
  float bias[8][4];
  {
    const int off = (ws - 1) * 2 * ws;
    const int cr[2] = {code_s[r0] + off, code_s[r1] + off};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int r = (e < 2) ? r0 : r1, c = j * 8 + 2 * t4 + (e & 1);
        float v = 0.f;
        if (r < T && c < T) {
          const int idx = cr[e >> 1] - code_s[c];
          v = a.table_f32 ? ((const float*)a.table)[idx * a.heads + h]
                          : __bfloat162float(((const __nv_bfloat16*)a.table)[idx * a.heads + h]);
        } else if (c >= T) {
          v = -INFINITY;                          // padded key columns never contribute
        }
        bias[j][e] = v;
      }
    }
  }
  __syncthreads();

  const AttnOperand* ops[3] = {&a.q, &a.k, &a.v};
  auto load_window = [&](int n, int b) {
#pragma unroll
    for (int m = 0; m < 3; ++m) {
      const AttnOperand& o = *ops[m];
      const __nv_bfloat16* src = (const __nv_bfloat16*)o.ptr + (long long)n * o.sn + (long long)h * o.sh;
      __nv_bfloat16* dst = &bufs[b][m][0];
      if (o.se == 1) {
        constexpr int VPR = D / 8;
        for (int i = tid; i < T * VPR; i += 128) {
          const int t = i / VPR, c = i - t * VPR;
          cp_async16(dst + t * RS + c * 8, src + (long long)t * o.st + c * 8);
        }
      } else {                                  // element-strided operand (e.g. a materialised K^T)
        for (int i = tid; i < T * D; i += 128) {
          const int e = i / T, t = i - e * T;
          dst[t * RS + e] = src[(long long)t * o.st + (long long)e * o.se];
        }
      }
    }
    if (a.shift > 0 && tid < TP) {
      const int wl = n - (int)fd_div((uint32_t)n, a.fd_wpi) * a.win_per_img;
      const int wy = (int)fd_div((uint32_t)wl, a.fd_nww), wx = wl - wy * a.nWw;
      lab_s[b][tid] = region_label2(my_ty, my_tx, ws, wy, wx, a.H, a.W, a.shift);
    }
  };

  int it = 0;
  if (cidx < a.n_windows) load_window(cidx, 0);
  cp_async_commit();
  for (int n = cidx; n < a.n_windows; n += cstride, ++it) {
    const int b = it & 1;
    if (n + cstride < a.n_windows) load_window(n + cstride, b ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (warp_active) {
      const uint32_t* Qw = reinterpret_cast<const uint32_t*>(&bufs[b][0][0]);
      const uint32_t* Kw = reinterpret_cast<const uint32_t*>(&bufs[b][1][0]);
      const __nv_bfloat16* Vs = &bufs[b][2][0];
      // ---- S = Q K^T -----------------------------------------------------------------------
      float s[8][4];
#pragma unroll
      for (int j = 0; j < 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        uint32_t af[4];
        af[0] = Qw[r0 * RW + kk * 8 + t4];
        af[1] = Qw[r1 * RW + kk * 8 + t4];
        af[2] = Qw[r0 * RW + kk * 8 + 4 + t4];
        af[3] = Qw[r1 * RW + kk * 8 + 4 + t4];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (j * 8 < T) {
            const uint32_t b0 = Kw[(j * 8 + g) * RW + kk * 8 + t4];
            const uint32_t b1 = Kw[(j * 8 + g) * RW + kk * 8 + 4 + t4];
            ptx::mma_m16n8k16_bf16(s[j], af, b0, b1);
          }
        }
      }
      // ---- scale + bias (+ mask on the windows that touch the seam), softmax ------------------
#pragma unroll
      for (int j = 0; j < 8; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) s[j][e] = fmaf(s[j][e], a.scale, bias[j][e]);
      }
      bool masked = false;
      if (a.shift > 0) {
        const int wl = n - (int)fd_div((uint32_t)n, a.fd_wpi) * a.win_per_img;
        const int wy = (int)fd_div((uint32_t)wl, a.fd_nww), wx = wl - wy * a.nWw;
        masked = (wy == a.nWh - 1) || (wx == a.nWw - 1);
      }
      if (masked) {
        const int l0 = lab_s[b][r0], l1 = lab_s[b][r1];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int lc = lab_s[b][j * 8 + 2 * t4 + e];
            if (l0 != lc) s[j][e] -= 100.f;
            if (l1 != lc) s[j][2 + e] -= 100.f;
          }
        }
      }
      float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        m0 = fmaxf(m0, fmaxf(s[j][0], s[j][1]));
        m1 = fmaxf(m1, fmaxf(s[j][2], s[j][3]));
      }
      m0 = fmaxf(m0, __shfl_xor_sync(0xFFFFFFFFu, m0, 1));
      m0 = fmaxf(m0, __shfl_xor_sync(0xFFFFFFFFu, m0, 2));
      m1 = fmaxf(m1, __shfl_xor_sync(0xFFFFFFFFu, m1, 1));
      m1 = fmaxf(m1, __shfl_xor_sync(0xFFFFFFFFu, m1, 2));
      float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float p0 = __expf(s[j][e] - m0), p1 = __expf(s[j][2 + e] - m1);
          s[j][e] = p0;
          s[j][2 + e] = p1;
          sum0 += p0;
          sum1 += p1;
        }
      }
      sum0 += __shfl_xor_sync(0xFFFFFFFFu, sum0, 1);
      sum0 += __shfl_xor_sync(0xFFFFFFFFu, sum0, 2);
      sum1 += __shfl_xor_sync(0xFFFFFFFFu, sum1, 1);
      sum1 += __shfl_xor_sync(0xFFFFFFFFu, sum1, 2);
      // ---- O = P V: the score fragments are the A fragments of the second MMA -----------------
      float o[D / 8][4];
#pragma unroll
      for (int j = 0; j < D / 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        if (kk * 16 < T) {
          uint32_t af[4];
          af[0] = float2_to_bf16x2(s[2 * kk][0], s[2 * kk][1]);
          af[1] = float2_to_bf16x2(s[2 * kk][2], s[2 * kk][3]);
          af[2] = float2_to_bf16x2(s[2 * kk + 1][0], s[2 * kk + 1][1]);
          af[3] = float2_to_bf16x2(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
          for (int j = 0; j < D / 8; ++j) {
            // V^T fragments by transposing 8x8 blocks of row-major V on the way out of shared memory
            uint32_t b0, b1;
            const __nv_bfloat16* rowp = Vs + (kk * 16 + (lane & 15)) * RS + j * 8;
            asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];"
                         : "=r"(b0), "=r"(b1)
                         : "r"(ptx::smem_u32(rowp)));
            ptx::mma_m16n8k16_bf16(o[j], af, b0, b1);
          }
        }
      }
      // stage this warp's 16 x D result over the q rows it alone consumed, then store whole rows
      const float inv0 = 1.f / sum0, inv1 = 1.f / sum1;
      uint32_t* Ow = reinterpret_cast<uint32_t*>(&bufs[b][0][0]);
      __syncwarp();
#pragma unroll
      for (int j = 0; j < D / 8; ++j) {
        Ow[r0 * RW + j * 4 + t4] = float2_to_bf16x2(o[j][0] * inv0, o[j][1] * inv0);
        Ow[r1 * RW + j * 4 + t4] = float2_to_bf16x2(o[j][2] * inv1, o[j][3] * inv1);
      }
      __syncwarp();
      __nv_bfloat16* dst = (__nv_bfloat16*)a.o.ptr + (long long)n * a.o.sn + (long long)h * a.o.sh;
      constexpr int VPR = D / 8;
      for (int i = lane; i < 16 * VPR; i += 32) {
        const int t = warp * 16 + i / VPR, c = i % VPR;
        if (t < T)
          *reinterpret_cast<uint4*>(dst + (long long)t * a.o.st + c * 8) =
              *reinterpret_cast<const uint4*>(&bufs[b][0][0] + t * RS + c * 8);
      }
    }
    __syncthreads();                            // buffer b is free for the prefetch after next
  }
  cp_async_wait<0>();
}

// fp32 variant (plain FMA): one CTA per (window, head); scores live in shared memory.
__global__ void __launch_bounds__(128) win_attn_f32_kernel(const __grid_constant__ WinAttnArgs a) {
  pdl_wait();
  pdl_launch_dependents();
  constexpr int DM = 32;
  __shared__ float Qs[TP * (DM + 1)], Ks[TP * (DM + 1)], Vs[TP * (DM + 1)];
  __shared__ float Ss[TP * (TP + 1)];
  __shared__ float tab_s[256];
  __shared__ int lab_s[TP];
  const int unit = blockIdx.x;
  const int n = unit / a.heads, h = unit - n * a.heads;
  const int T = a.T, ws = a.ws, D = a.d;
  const int tid = threadIdx.x;
  const AttnOperand* ops[3] = {&a.q, &a.k, &a.v};
  float* dsts[3] = {Qs, Ks, Vs};
  for (int m = 0; m < 3; ++m) {
    const float* src = unit_ptr<float>(*ops[m], n, h);
    for (int i = tid; i < T * D; i += 128) {
      int t, e;
      if (ops[m]->se == 1) { t = i / D; e = i - t * D; } else { e = i / T; t = i - e * T; }
      dsts[m][t * (DM + 1) + e] = src[(long long)t * ops[m]->st + (long long)e * ops[m]->se];
    }
  }
  const int nb = (2 * ws - 1) * (2 * ws - 1);
  for (int i = tid; i < nb; i += 128)
    tab_s[i] = a.table_f32 ? ((const float*)a.table)[i * a.heads + h]
                           : __bfloat162float(((const __nv_bfloat16*)a.table)[i * a.heads + h]);
  if (tid < TP) {
    int lab = 0;
    if (a.shift > 0 && tid < T) {
      const int wl = n % a.win_per_img;
      lab = region_label(tid, ws, wl / a.nWw, wl % a.nWw, a.H, a.W, a.shift);
    }
    lab_s[tid] = lab;
  }
  __syncthreads();
  for (int idx = tid; idx < T * T; idx += 128) {
    const int i = idx / T, j = idx - i * T;
    float acc = 0.f;
    for (int e = 0; e < D; ++e) acc = fmaf(Qs[i * (DM + 1) + e], Ks[j * (DM + 1) + e], acc);
    const int bi = (i / ws - j / ws + ws - 1) * (2 * ws - 1) + (i % ws - j % ws + ws - 1);
    Ss[i * (TP + 1) + j] = acc * a.scale + tab_s[bi] + (lab_s[i] != lab_s[j] ? -100.f : 0.f);
  }
  __syncthreads();
  // softmax: one warp per row, shuffle reductions
  const int warp = tid >> 5, lane = tid & 31;
  for (int i = warp; i < T; i += 4) {
    float m = -INFINITY;
    for (int j = lane; j < T; j += 32) m = fmaxf(m, Ss[i * (TP + 1) + j]);
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    float sum = 0.f;
    for (int j = lane; j < T; j += 32) {
      const float p = expf(Ss[i * (TP + 1) + j] - m);
      Ss[i * (TP + 1) + j] = p;
      sum += p;
    }
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
    const float inv = 1.f / sum;
    for (int j = lane; j < T; j += 32) Ss[i * (TP + 1) + j] *= inv;
  }
  __syncthreads();
  float* dst = (float*)a.o.ptr + (long long)n * a.o.sn + (long long)h * a.o.sh;
  for (int idx = tid; idx < T * D; idx += 128) {
    const int i = idx / D, e = idx - i * D;
    float acc = 0.f;
    for (int j = 0; j < T; ++j) acc = fmaf(Ss[i * (TP + 1) + j], Vs[j * (DM + 1) + e], acc);
    dst[(long long)i * a.o.st + e] = acc;
  }
}

}  // namespace

int launch_window_attention(const WinAttnArgs& a, int dtype, long long n_windows, cudaStream_t st) {
  if (a.T < 1 || a.T > TP || a.ws * a.ws != a.T || (2 * a.ws - 1) * (2 * a.ws - 1) > 256) return SMARTMEM_ERR_UNSUPPORTED;
  long long units = n_windows * a.heads;
  if (units < 1 || units >= (1ll << 31)) return SMARTMEM_ERR_UNSUPPORTED;
  if (dtype == SMARTMEM_F32) {
    if (a.d > 32) return SMARTMEM_ERR_UNSUPPORTED;
    profile_tick("window_attention_f32", st);
    launch_pdl(win_attn_f32_kernel, dim3((unsigned)units), dim3(128), 0, st, a);
  } else {
    // vector loads need 16-byte aligned rows when the element stride is 1
    const AttnOperand* ops[3] = {&a.q, &a.k, &a.v};
    for (auto* o : ops)
      if (o->se == 1 && (o->st % 8 || o->sn % 8 || o->sh % 8 || ((uintptr_t)o->ptr & 15))) return SMARTMEM_ERR_ALIGNMENT;
    if (a.o.se != 1 || a.o.st % 8 || a.o.sn % 8 || a.o.sh % 8 || ((uintptr_t)a.o.ptr & 15)) return SMARTMEM_ERR_ALIGNMENT;
    if (a.d != 16 && a.d != 32) return SMARTMEM_ERR_UNSUPPORTED;
    static const bool legacy = [] { const char* e = getenv("SMARTMEM_WINDOW_LEGACY"); return e && e[0] == '1'; }();
    if (!legacy) {
      const int rc = launch_window_attention_tc(a, n_windows, st);
      if (rc != SMARTMEM_ERR_UNSUPPORTED) return rc;
    }
    WinAttnArgs b = a;
    b.n_windows = (int)n_windows;
    b.nWh = a.win_per_img / a.nWw;
    b.fd_wpi = make_fastdiv((uint32_t)a.win_per_img);
    b.fd_nww = make_fastdiv((uint32_t)a.nWw);
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) sms = 148;
    long long per_head = (long long)sms * 5 / a.heads;           // ~5 resident CTAs per SM
    if (per_head < 1) per_head = 1;
    if (per_head > n_windows) per_head = n_windows;
    const unsigned grid = (unsigned)(per_head * a.heads);
    profile_tick("window_attention", st);
    if (a.d == 32) launch_pdl(win_attn_bf16_kernel<32>, dim3(grid), dim3(128), 0, st, b);
    else launch_pdl(win_attn_bf16_kernel<16>, dim3(grid), dim3(128), 0, st, b);
  }
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

}  // namespace smartmem
