// Host-side interface of the attention kernels and the fp32 plain-FMA GEMM.
#pragma once
#include "common.cuh"

namespace smartmem {

// An attention operand x[n, h, t, e] addressed as ptr + n*sn + h*sh + t*st + e*se (elements).
struct AttnOperand {
  const void* ptr;
  long long sn, sh, st, se;
};

struct WinAttnArgs {
  AttnOperand q, k, v, o;
  const void* table;        // [(2ws-1)^2, heads]
  int table_f32;
  int heads, T, ws, d, shift, H, W, nWw, win_per_img;
  int n_windows, nWh;       // set by the launcher
  FastDiv fd_wpi, fd_nww;   // reciprocals of win_per_img and nWw (set by the launcher)
  float scale;
};
int launch_window_attention(const WinAttnArgs& a, int dtype, long long n_windows, cudaStream_t st);
int launch_window_attention_tc(const WinAttnArgs& a, long long n_windows, cudaStream_t st);

#ifdef __CUDACC__
// Region label of token (ty, tx) of window (wy, wx) of a shifted block, in shifted coordinates:
// 3 * r(row) + r(col) with r = 0 before the last window, 1 in its unwrapped part, 2 in the wrapped part.
__device__ __forceinline__ int region_label2(int ty, int tx, int ws, int wy, int wx, int H, int W, int shift) {
  const int hp = wy * ws + ty, wp = wx * ws + tx;
  const int rh = hp < H - ws ? 0 : (hp < H - shift ? 1 : 2);
  const int rw = wp < W - ws ? 0 : (wp < W - shift ? 1 : 2);
  return 3 * rh + rw;
}
#endif

// Causal attention over [S] positions for `heads` heads of dimension 128 (bf16).
struct CausalAttnArgs {
  AttnOperand q, k, v, o;   // n = batch, h = head
  int S, heads, batch;
  float scale;
};
int launch_causal_attention(const CausalAttnArgs& a, cudaStream_t st);
// Rotary embedding: (cos, sin) table [S, head_dim/2] as float2, and the stand-alone in-place
// rotation of rows [rows, head_dim] (position = row % S) used by the explicit variant.  With a partial
// rotary dimension R the table is built for "head_dim" = R and only the first R elements of a row rotate.
int launch_rope_table(float* tab, int S, int head_dim, float theta, cudaStream_t st);
int launch_rope_rows(void* x, long long rows, int S, int head_dim, const float* tab, cudaStream_t st, int rotary_dim = 0);

// out[M,N] = A[M,K] W[N,K]^T (+bias)(GELU)(+residual), fp32 with plain FMAs.  Rows of A may be
// gathered through `amap`, rows of out scattered through `omap` (residual uses the same offsets).
struct SimtGemmArgs {
  const float* A; const float* W; const float* bias; const float* residual; float* out;
  int M, N, K;
  long long lda, ldc;
  int gelu, has_amap, has_omap;
  DevMap amap, omap;
};
int launch_gemm_simt_f32(const SimtGemmArgs& a, cudaStream_t st);

}  // namespace smartmem
