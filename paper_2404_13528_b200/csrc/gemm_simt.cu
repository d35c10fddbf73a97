// fp32 GEMM with plain FMAs for the fp32 configuration: the tf32 tensor-core path keeps 10
// mantissa bits and cannot stay within 1e-4 of an fp64 reference, so fp32 inputs take this
// kernel.  It supports the same folded index maps as the tensor-core path: rows of A
// gathered through a map, rows of the result scattered through a map.
#include "attn.cuh"

namespace smartmem {
namespace {

__global__ void __launch_bounds__(256) gemm_simt_f32_kernel(const __grid_constant__ SimtGemmArgs g) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ float As[16][17], Ws[16][17];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int row = blockIdx.y * 16 + ty, col = blockIdx.x * 16 + tx;
  const int wrow = blockIdx.x * 16 + ty;
  long long aoff = 0;
  if (row < g.M) aoff = g.has_amap ? devmap_eval(g.amap, (uint32_t)row) : (long long)row * g.lda;
  float acc = 0.f;
  for (int k0 = 0; k0 < g.K; k0 += 16) {
    As[ty][tx] = (row < g.M && k0 + tx < g.K) ? g.A[aoff + k0 + tx] : 0.f;
    Ws[ty][tx] = (wrow < g.N && k0 + tx < g.K) ? g.W[(long long)wrow * g.K + k0 + tx] : 0.f;
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) acc = fmaf(As[ty][k], Ws[tx][k], acc);
    __syncthreads();
  }
  if (row >= g.M || col >= g.N) return;
  if (g.bias) acc += g.bias[col];
  if (g.gelu) acc = gelu_erf(acc);
  const long long ooff = (g.has_omap ? devmap_eval(g.omap, (uint32_t)row) : (long long)row * g.ldc) + col;
  if (g.residual) acc += g.residual[ooff];
  g.out[ooff] = acc;
}

}  // namespace

int launch_gemm_simt_f32(const SimtGemmArgs& a, cudaStream_t st) {
  if (a.M < 1 || a.N < 1 || a.K < 1) return SMARTMEM_ERR_UNSUPPORTED;
  dim3 grid((a.N + 15) / 16, (a.M + 15) / 16);
  if (grid.y > 65535) return SMARTMEM_ERR_UNSUPPORTED;
  profile_tick("gemm_simt_f32", st);
  launch_pdl(gemm_simt_f32_kernel, dim3(grid), dim3(256), 0, st, a);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

}  // namespace smartmem
