// Host-side interface of the tcgen05 GEMM.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace smartmem {

// A [rows, K] bf16 operand as it lies in the producer's buffer: its rows are indexed by up
// to 3 "row atoms" (mixed radix, outermost first) below up to 3 batch atoms; strides are in
// elements.  k_stride == 1: reduction-dim contiguous (K-major).  Otherwise the innermost row
// atom must be contiguous (MN-major operand).
struct TcOperand {
  const void* ptr;
  int n_batch_atoms, n_row_atoms;
  long long batch_extent[3], batch_stride[3];
  long long row_extent[3], row_stride[3];
  long long K, k_stride;
};

struct TcEpilogue {
  void* out;                 // bf16
  long long ldc;             // row pitch in elements (ignored for rows placed by rowmap)
  long long out_batch_stride;
  const void* bias;          // [N] bf16 or null
  const void* residual;      // same addressing as out, or null
  int gelu;
  const DevMap* rowmap;      // output row -> element offset, or null
  int rope_cols, rope_S;     // rotate columns [0, rope_cols) in 128-wide heads; position = rope_pos0 + row % rope_S
  float rope_log2_theta;     // angle of pair i at position p: p * 2^(-i/64 * rope_log2_theta)
  int rope_pos0;
  int rope_dim;              // rotary dimension R in {32, 64, 128} (0 = 128): only the first R columns of a head rotate,
                             // in pairs (i, i + R/2), pair i at angle p * 2^(-i/(R/2) * rope_log2_theta)
  // Column-segmented output (seg_cols > 0, a multiple of 256; no rowmap, residual or batch): columns
  // [s*seg_cols, (s+1)*seg_cols) of row r go to seg_out[s] + r*seg_ld[s] (elements), s < 3.  `out`
  // and `ldc` are ignored.  Lets one GEMM store into several destinations of different pitch.
  int seg_cols;
  void* seg_out[3];
  long long seg_ld[3];
  // Second copy of the result (null: none) for a consumer whose reduction dimension is the row index inside groups of
  // out2_S rows: element (row, col) also goes to out2[(row / out2_S) * N * out2_S + col * out2_S + row % out2_S].
  // batch == 1, M a multiple of out2_S.
  void* out2;
  long long out2_S;
};

int tc_operand_from_map(const smartmem_index_map_t& m, int n_batch_atoms, int n_row_atoms, const void* ptr,
                        TcOperand* op);
TcOperand tc_operand_plain(const void* ptr, long long rows, long long K, long long ld);
int launch_gemm_tc(const TcOperand& A, const TcOperand& B, const TcEpilogue& ep, long long batch, long long M,
                   long long N, long long K, cudaStream_t st);

// bf16 row-major [outer, inner] matrix as a 2-D tensor map with 128-byte swizzle (box_inner = 64).
int tc_encode_2d(const void* ptr, long long inner, long long outer, long long pitch_elems, int box_inner, int box_outer,
                 CUtensorMap* out);
// Same with 64-byte swizzle: boxes of 32 bf16 columns (64-byte rows).
int tc_encode_2d_sw64(const void* ptr, long long inner, long long outer, long long pitch_elems, int box_inner,
                      int box_outer, CUtensorMap* out);
// bf16 tensor of `rank` dimensions (innermost first; strides in elements for dimensions 1..rank-1) with 64-byte swizzle and a box
// of 32 innermost elements.
int tc_encode_nd_sw64(const void* ptr, int rank, const long long* dims, const long long* strides_elems, const int* box,
                      CUtensorMap* out);
int tc_sm_count();

// Fused MLP half of a block: out = A + GELU(LN(A) W1^T + b1) W2^T + b2 with the hidden activation and the
// normalised rows kept on chip.  A [M, C], W1 [hidden, C], W2 [C, hidden], C in {64, 96}, hidden a multiple
// of 128 with both weight matrices fitting shared memory; ln_gamma/ln_beta [C]: LayerNorm over C, eps inside
// the square root.  out may not alias A.
bool mlp_fused_supported(long long C, long long hidden);
int launch_mlp_fused(const void* A, const void* ln_gamma, const void* ln_beta, float ln_eps, const void* W1, const void* b1,
                     const void* W2, const void* b2, void* out, long long M, long long C, long long hidden,
                     cudaStream_t st);

// LayerNorm o row-gather o linear for narrow rows: out[m, :] = LN(X[src(m), :]) W^T + bias, with X rows of
// K in {64, 96} elements, W [N, K], N a multiple of 96 (at most 288).  `rowmap` (null: identity) gives
// the element offset of consumer row m in X; gamma/beta null: no normalisation (plain gather).
bool gemm_ln_supported(long long N, long long K);
int launch_gemm_ln(const void* X, const DevMap* rowmap, const void* gamma, const void* beta, float eps, const void* W,
                   const void* bias, void* out, long long M, long long N, long long K, cudaStream_t st);

// Attention half of a narrow Swin block (bf16, head dimension 32, 2 or 3 heads, window^2 <= 64) in one kernel:
// y = x + unshift(unpartition(proj(window_attention(qkv(LN1(partition(shift(x)))))))), every layout operator folded into the
// row gather / row scatter through `rowmap` (windowed row -> element offset of the token in x and y).  x and y must not alias.
bool swin_attn_fused_supported(int dtype, int C, int heads, int window);
int launch_swin_attn_fused(const smartmem_swin_params_t& p, const DevMap& rowmap, const void* x, void* y, cudaStream_t st);

}  // namespace smartmem
