// LayerNorm / RMSNorm over the last dimension (kept operators: ILD & Variable, Table 3).
// The rows may be fetched through a composed index map (cyclic shift + window partition
// folded into the loads), so the normalised rows come out in the consumer's order with no
// layout copy in between.  Statistics are fp32 and two-pass (mean, then centred variance);
// reductions use warp shuffles.
#include "common.cuh"

namespace smartmem {
namespace {

template <int LPR>
__device__ __forceinline__ float group_sum(float v) {
#pragma unroll
  for (int o = LPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// LPR lanes cooperate on one row and keep up to 4 16-byte vectors each in registers (vector k of
// lane l is vector l + k * LPR of the row, so a warp-wide load covers 32 / LPR rows with runs of
// LPR * 16 contiguous bytes).  RPG rows per lane group are in flight together.  GENERIC: any row
// length; the row is re-read from L1/L2 for each pass instead of being kept.
template <typename T, int LPR, bool RMS, int RPG, bool GENERIC>
__global__ void __launch_bounds__(256) norm_kernel(const T* __restrict__ src, T* __restrict__ dst,
                                                   const T* __restrict__ gamma, const T* __restrict__ beta, float eps,
                                                   long long rows, int C, int vpl, const __grid_constant__ DevMap rowmap,
                                                   int has_map) {
  constexpr int KV = ElemIO<T>::kVec;
  constexpr int NV = GENERIC ? 1 : 4;
  constexpr int GPB = 8 * (32 / LPR);                       // lane groups per block
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int sub = lane % LPR, grp = warp * (32 / LPR) + lane / LPR;
  const long long row0 = (long long)blockIdx.x * (GPB * RPG) + grp;
  const int nvec = C / KV;
  const float invC = 1.0f / (float)C;
  float v[RPG][NV][KV];
  const T* s[RPG];
  bool active[RPG];
  float sum[RPG];
  pdl_wait();
  pdl_launch_dependents();
#pragma unroll
  for (int r = 0; r < RPG; ++r) {
    const long long row = row0 + (long long)r * GPB;
    active[r] = row < rows;
    long long soff = 0;
    if (has_map) {
      if (sub == 0 && active[r]) soff = devmap_eval_unrolled(rowmap, (uint32_t)row);   // one lane per row, then broadcast
      soff = __shfl_sync(0xFFFFFFFFu, soff, lane - sub);
    } else if (active[r]) {
      soff = row * (long long)C;
    }
    s[r] = src + soff;
  }
#pragma unroll
  for (int r = 0; r < RPG; ++r) {
    sum[r] = 0.f;
    if constexpr (!GENERIC) {
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        const int vi = sub + k * LPR;
        if (k < vpl && active[r] && vi < nvec) {
          ElemIO<T>::load(s[r] + vi * KV, v[r][k]);
        } else {
#pragma unroll
          for (int e = 0; e < KV; ++e) v[r][k][e] = 0.f;
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < RPG; ++r) {
    if constexpr (!GENERIC) {
#pragma unroll
      for (int k = 0; k < NV; ++k)
        if (k < vpl) {
#pragma unroll
          for (int e = 0; e < KV; ++e) sum[r] += RMS ? v[r][k][e] * v[r][k][e] : v[r][k][e];
        }
    } else {
      for (int vi = sub; vi < nvec && active[r]; vi += LPR) {
        ElemIO<T>::load(s[r] + vi * KV, v[r][0]);
#pragma unroll
        for (int e = 0; e < KV; ++e) sum[r] += RMS ? v[r][0][e] * v[r][0][e] : v[r][0][e];
      }
    }
    sum[r] = group_sum<LPR>(sum[r]);
  }
  float mean[RPG], rstd[RPG];
#pragma unroll
  for (int r = 0; r < RPG; ++r) {
    mean[r] = 0.f;
    if constexpr (RMS) {
      rstd[r] = rsqrtf(sum[r] * invC + eps);
    } else {
      mean[r] = sum[r] * invC;
      float sq = 0.f;
      if constexpr (!GENERIC) {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
          const int vi = sub + k * LPR;
          if (k < vpl && active[r] && vi < nvec) {
#pragma unroll
            for (int e = 0; e < KV; ++e) sq += (v[r][k][e] - mean[r]) * (v[r][k][e] - mean[r]);
          }
        }
      } else {
        for (int vi = sub; vi < nvec && active[r]; vi += LPR) {
          ElemIO<T>::load(s[r] + vi * KV, v[r][0]);
#pragma unroll
          for (int e = 0; e < KV; ++e) sq += (v[r][0][e] - mean[r]) * (v[r][0][e] - mean[r]);
        }
      }
      sq = group_sum<LPR>(sq);
      rstd[r] = rsqrtf(sq * invC + eps);
    }
  }
  // y = x * (rstd g) + (beta - mean rstd g): two fused multiply-adds per element
  auto emit = [&](int r, int vi, float* x, const float* g, const float* b) {
    float y[KV];
    const float ms = -mean[r] * rstd[r];
#pragma unroll
    for (int e = 0; e < KV; ++e) y[e] = RMS ? x[e] * rstd[r] * g[e] : fmaf(fmaf(x[e], rstd[r], ms), g[e], b[e]);
    ElemIO<T>::store(dst + (row0 + (long long)r * GPB) * (long long)C + vi * KV, y);
  };
  if constexpr (!GENERIC) {
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      const int vi = sub + k * LPR;
      if (k < vpl && vi < nvec) {
        float g[KV], b[KV];
        ElemIO<T>::load(gamma + vi * KV, g);
        if constexpr (!RMS) ElemIO<T>::load(beta + vi * KV, b);
#pragma unroll
        for (int r = 0; r < RPG; ++r)
          if (active[r]) emit(r, vi, v[r][k], g, b);
      }
    }
  } else {
    for (int vi = sub; vi < nvec; vi += LPR) {
      float g[KV], b[KV];
      ElemIO<T>::load(gamma + vi * KV, g);
      if constexpr (!RMS) ElemIO<T>::load(beta + vi * KV, b);
#pragma unroll
      for (int r = 0; r < RPG; ++r)
        if (active[r]) {
          ElemIO<T>::load(s[r] + vi * KV, v[r][0]);
          emit(r, vi, v[r][0], g, b);
        }
    }
  }
}

// Wide rows (more than 128 vectors): one CTA per row, every thread keeps up to 4 of the row's 16-byte
// vectors in registers, so the whole row is requested at once (the generic kernel above walks a
// row one vector per lane at a time and is bound by that chain of load latencies).
template <typename T, bool RMS>
__global__ void __launch_bounds__(256) norm_wide_kernel(const T* __restrict__ src, T* __restrict__ dst,
                                                        const T* __restrict__ gamma, const T* __restrict__ beta, float eps,
                                                        int C) {
  constexpr int KV = ElemIO<T>::kVec;
  constexpr int NVW = 4;
  __shared__ float red[8];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = C / KV;
  const float invC = 1.0f / (float)C;
  auto block_sum = [&](float x) {
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, m);
    __syncthreads();                                       // the previous round's reads of red[] are done
    if (lane == 0) red[warp] = x;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) t += red[w];
    return t;
  };
  pdl_wait();
  pdl_launch_dependents();
  const T* s = src + (long long)blockIdx.x * C;
  T* d = dst + (long long)blockIdx.x * C;
  float v[NVW][KV];
#pragma unroll
  for (int k = 0; k < NVW; ++k) {
    const int vi = tid + k * 256;
    if (vi < nvec) {
      ElemIO<T>::load(s + vi * KV, v[k]);
    } else {
#pragma unroll
      for (int e = 0; e < KV; ++e) v[k][e] = 0.f;
    }
  }
  float sum = 0.f;
#pragma unroll
  for (int k = 0; k < NVW; ++k)
#pragma unroll
    for (int e = 0; e < KV; ++e) sum += RMS ? v[k][e] * v[k][e] : v[k][e];
  sum = block_sum(sum);
  float mean = 0.f, rstd;
  if constexpr (RMS) {
    rstd = rsqrtf(sum * invC + eps);
  } else {
    mean = sum * invC;
    float sq = 0.f;
#pragma unroll
    for (int k = 0; k < NVW; ++k)
      if (tid + k * 256 < nvec) {
#pragma unroll
        for (int e = 0; e < KV; ++e) sq += (v[k][e] - mean) * (v[k][e] - mean);
      }
    sq = block_sum(sq);
    rstd = rsqrtf(sq * invC + eps);
  }
  const float ms = -mean * rstd;
#pragma unroll
  for (int k = 0; k < NVW; ++k) {
    const int vi = tid + k * 256;
    if (vi < nvec) {
      float g[KV], b[KV], y[KV];
      ElemIO<T>::load(gamma + vi * KV, g);
      if constexpr (!RMS) ElemIO<T>::load(beta + vi * KV, b);
#pragma unroll
      for (int e = 0; e < KV; ++e) y[e] = RMS ? v[k][e] * rstd * g[e] : fmaf(fmaf(v[k][e], rstd, ms), g[e], b[e]);
      ElemIO<T>::store(d + vi * KV, y);
    }
  }
}

// Rows whose elements are fetched through an eliminated layout chain: vector u of the consumer's
// [rows, C] tensor (16 bytes, never straddling a contiguous run of the producer) lies at element
// offset map(u).  One warp per RPW rows, NV vectors per lane and row in registers; the result is
// written contiguously.
template <typename T, bool RMS, int NV, int RPW>
__global__ void __launch_bounds__(256) norm_gather_kernel(const T* __restrict__ src, T* __restrict__ dst,
                                                          const T* __restrict__ gamma, const T* __restrict__ beta, float eps,
                                                          long long rows, int C, const __grid_constant__ DevMap map) {
  constexpr int KV = ElemIO<T>::kVec;
  const int lane = threadIdx.x & 31;
  const long long row0 = ((long long)blockIdx.x * 8 + (threadIdx.x >> 5)) * RPW;
  const int nvec = C / KV;
  const float invC = 1.0f / (float)C;
  pdl_wait();
  pdl_launch_dependents();
  if (row0 >= rows) return;
  float v[RPW][NV][KV];
#pragma unroll
  for (int r = 0; r < RPW; ++r)
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      const int vi = lane + k * 32;
      if (vi < nvec && row0 + r < rows) {
        const long long off = devmap_eval_unrolled(map, (uint32_t)((row0 + r) * nvec + vi));
        ElemIO<T>::load(src + off, v[r][k]);
      } else {
#pragma unroll
        for (int e = 0; e < KV; ++e) v[r][k][e] = 0.f;
      }
    }
  float mean[RPW], rstd[RPW];
#pragma unroll
  for (int r = 0; r < RPW; ++r) {
    float sum = 0.f;
#pragma unroll
    for (int k = 0; k < NV; ++k)
#pragma unroll
      for (int e = 0; e < KV; ++e) sum += RMS ? v[r][k][e] * v[r][k][e] : v[r][k][e];
    sum = group_sum<32>(sum);
    mean[r] = 0.f;
    if constexpr (RMS) {
      rstd[r] = rsqrtf(sum * invC + eps);
    } else {
      mean[r] = sum * invC;
      float sq = 0.f;
#pragma unroll
      for (int k = 0; k < NV; ++k)
        if (lane + k * 32 < nvec) {
#pragma unroll
          for (int e = 0; e < KV; ++e) sq += (v[r][k][e] - mean[r]) * (v[r][k][e] - mean[r]);
        }
      sq = group_sum<32>(sq);
      rstd[r] = rsqrtf(sq * invC + eps);
    }
  }
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    const int vi = lane + k * 32;
    if (vi < nvec) {
      float g[KV], b[KV];
      ElemIO<T>::load(gamma + vi * KV, g);
      if constexpr (!RMS) ElemIO<T>::load(beta + vi * KV, b);
#pragma unroll
      for (int r = 0; r < RPW; ++r)
        if (row0 + r < rows) {
          float y[KV];
          const float ms = -mean[r] * rstd[r];
#pragma unroll
          for (int e = 0; e < KV; ++e) y[e] = RMS ? v[r][k][e] * rstd[r] * g[e] : fmaf(fmaf(v[r][k][e], rstd[r], ms), g[e], b[e]);
          ElemIO<T>::store(dst + (row0 + r) * (long long)C + vi * KV, y);
        }
    }
  }
}

template <typename T, bool RMS>
int launch_norm_t(const void* src, void* dst, const void* gamma, const void* beta, float eps, long long rows, int C,
                  const DevMap* rowmap, cudaStream_t st) {
  constexpr int KV = ElemIO<T>::kVec;
  if (C % KV) return SMARTMEM_ERR_UNSUPPORTED;
  if (rows >= (1ll << 31)) return SMARTMEM_ERR_UNSUPPORTED;
  const int nvec = C / KV;
  DevMap dm;
  memset(&dm, 0, sizeof(dm));
  if (rowmap) dm = *rowmap;
  const int has = rowmap ? 1 : 0;
  const T* s = (const T*)src;
  T* d = (T*)dst;
  const T* g = (const T*)gamma;
  const T* b = (const T*)beta;
#define SM_LAUNCH(LPR, RPG, GEN)                                                                          \
  {                                                                                                       \
    const int vpl = (nvec + LPR - 1) / LPR;                                                               \
    long long rpb = 8 * (32 / LPR) * RPG;                                                                 \
    unsigned grid = (unsigned)((rows + rpb - 1) / rpb);                                                   \
    launch_pdl(norm_kernel<T, LPR, RMS, RPG, GEN>, dim3(grid), dim3(256), 0, st, s, d, g, b, eps, rows, C, vpl, dm, has);     \
  }
  if (nvec <= 16) SM_LAUNCH(4, 1, false)
  else if (nvec <= 32) SM_LAUNCH(8, 2, false)
  else if (nvec <= 64) SM_LAUNCH(16, 1, false)
  else if (nvec <= 128) SM_LAUNCH(32, 1, false)
  else if (!rowmap && nvec <= 1024)
    launch_pdl(norm_wide_kernel<T, RMS>, dim3((unsigned)rows), dim3(256), 0, st, s, d, g, b, eps, C);
  else SM_LAUNCH(32, 1, true)
#undef SM_LAUNCH
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

template <typename T>
int launch_norm_map_t(const void* src, void* dst, const void* gamma, const void* beta, float eps,
                      const smartmem_index_map_t& map, int C, cudaStream_t st) {
  constexpr int KV = ElemIO<T>::kVec;
  if (C % KV || C / KV > 128 || map.vec_elems != KV || map.klass == 3) return SMARTMEM_ERR_UNSUPPORTED;
  const long long rows = map.n_elements / C;
  if (map.n_elements / KV >= (1ll << 31)) return SMARTMEM_ERR_UNSUPPORTED;
  DevMap dm;
  if (!make_devmap(map, 0, map.n_atoms, KV, true, &dm)) return SMARTMEM_ERR_UNSUPPORTED;
  const int nvec = C / KV;
#define SM_NG(NV_, RPW_)                                                                                             \
  launch_pdl(norm_gather_kernel<T, false, NV_, RPW_>, dim3((unsigned)((rows + 8 * RPW_ - 1) / (8 * RPW_))), dim3(256), 0, st, \
             (const T*)src, (T*)dst, (const T*)gamma, (const T*)beta, eps, rows, C, dm);
  // one row per warp: two and four rows per warp were measured 1.2x and 1.8x slower (registers halve the resident warps)
  if (nvec <= 32) SM_NG(1, 1)
  else if (nvec <= 64) SM_NG(2, 1)
  else SM_NG(4, 1)
#undef SM_NG
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

}  // namespace

int launch_layernorm_map(int dtype, const void* src, void* dst, const void* gamma, const void* beta, float eps,
                         const smartmem_index_map_t& map, int C, cudaStream_t st) {
  profile_tick("layernorm_map", st);
  if (dtype == SMARTMEM_F32) return launch_norm_map_t<float>(src, dst, gamma, beta, eps, map, C, st);
  return launch_norm_map_t<__nv_bfloat16>(src, dst, gamma, beta, eps, map, C, st);
}

int launch_norm(int dtype, bool rms, const void* src, void* dst, const void* gamma, const void* beta, float eps,
                long long rows, int C, const DevMap* rowmap, cudaStream_t st) {
  profile_tick(rms ? "rmsnorm" : "layernorm", st);
  if (rows == 0) return SMARTMEM_OK;
  if (dtype == SMARTMEM_F32)
    return rms ? launch_norm_t<float, true>(src, dst, gamma, beta, eps, rows, C, rowmap, st)
               : launch_norm_t<float, false>(src, dst, gamma, beta, eps, rows, C, rowmap, st);
  return rms ? launch_norm_t<__nv_bfloat16, true>(src, dst, gamma, beta, eps, rows, C, rowmap, st)
             : launch_norm_t<__nv_bfloat16, false>(src, dst, gamma, beta, eps, rows, C, rowmap, st);
}

}  // namespace smartmem
