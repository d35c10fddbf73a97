// Shared-memory operand layouts and the LayerNorm-in-the-product helpers used by the fused
// tcgen05 kernels (attention half, MLP half).
//
// LayerNorm folded into the product that consumes it:
//   LN(x) W^T + b = rstd (x W'^T - mean c + sigma b'),   W' = bf16(gamma (.) W),  c_n = sum_k W'_nk,
//   b'_n = b_n + sum_k beta_k W_nk,  sigma = 1 / rstd.
// The raw rows go to the tensor core unchanged; the two rank-one terms ride on one extra k16 step
// whose operands hold -mean and sigma (row side) and c and b' (column side), each split into three
// bf16 pieces (24 significant bits), so that the accumulator only needs one multiply by rstd.
#pragma once
#include "common.cuh"

namespace smartmem {

// K-major tile of 64-byte rows with the 64-byte swizzle: 8-row groups 512 bytes apart
__device__ __forceinline__ uint64_t desc_sw64(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(16 >> 4) << 16;
  d |= (uint64_t)(512 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)4 << 61;
  return d;
}
// K-major tile without swizzle: 8 x 16-byte core matrices; the two of a k16 step 128 bytes apart, 8-row groups 256 bytes apart
__device__ __forceinline__ uint64_t desc_plain(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(128 >> 4) << 16;
  d |= (uint64_t)(256 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  return d;
}
__device__ __forceinline__ uint32_t plain_off(int row, int kc) { return (uint32_t)((row >> 3) * 256 + kc * 128 + (row & 7) * 16); }
// byte offset of 16-byte chunk `ch` (0..3) of row `row` inside a 64-byte-row tile with the 64-byte swizzle
__device__ __forceinline__ uint32_t sw64_off(int row, int ch) { return (uint32_t)(row * 64 + ((ch ^ ((row >> 1) & 3)) << 4)); }

// v = hi + mid + lo with three bf16 pieces (24 significant bits)
__device__ __forceinline__ void split3(float v, uint32_t& hi, uint32_t& mid, uint32_t& lo) {
  const __nv_bfloat16 a = __float2bfloat16_rn(v);
  const float r1 = v - __bfloat162float(a);
  const __nv_bfloat16 b = __float2bfloat16_rn(r1);
  const __nv_bfloat16 c = __float2bfloat16_rn(r1 - __bfloat162float(b));
  hi = __bfloat16_as_ushort(a); mid = __bfloat16_as_ushort(b); lo = __bfloat16_as_ushort(c);
}
// The extra k-step.  Operand side (per row): pieces of u = -mean and s = sigma; weight side (per column): pieces of c and b'.
// Position by position the products are  u_h c_h, u_h c_m, u_m c_h, u_h c_l, u_l c_h, u_m c_m  and the same for (s, b').
__device__ __forceinline__ void extra_row(float u, float s, uint4& k0, uint4& k1) {
  uint32_t uh, um, ul, sh, sm_, sl;
  split3(u, uh, um, ul);
  split3(s, sh, sm_, sl);
  k0 = make_uint4(uh | (uh << 16), um | (uh << 16), ul | (um << 16), sh | (sh << 16));
  k1 = make_uint4(sm_ | (sh << 16), sl | (sm_ << 16), 0x3F803F80u, 0x00003F80u);   // positions 12..14: ones (see bias_col)
}
// Weight side of a bias that rides on the same operand rows: positions 12..14 of a row hold ones, so a column whose
// positions 12..14 hold the three pieces of v (and zeros elsewhere) adds v to every row of the product.
__device__ __forceinline__ void bias_col(float v, uint4& k0, uint4& k1) {
  uint32_t h, m, l;
  split3(v, h, m, l);
  k0 = make_uint4(0u, 0u, 0u, 0u);
  k1 = make_uint4(0u, 0u, h | (m << 16), l);
}
__device__ __forceinline__ void extra_col(float c, float b, uint4& k0, uint4& k1) {
  uint32_t ch, cm, cl, bh, bm, bl;
  split3(c, ch, cm, cl);
  split3(b, bh, bm, bl);
  k0 = make_uint4(ch | (cm << 16), ch | (cl << 16), ch | (cm << 16), bh | (bm << 16));
  k1 = make_uint4(bh | (bl << 16), bh | (bm << 16), 0u, 0u);
}

}  // namespace smartmem
