// LayerNorm / RMSNorm over the last dimension (kept operators: ILD & Variable, Table 3).
// The rows may be fetched through a composed index map (cyclic shift + window partition
// folded into the loads), so the normalised rows come out in the consumer's order with no
// layout copy in between.  Statistics are fp32 and two-pass (mean, then centred variance);
// reductions use warp shuffles.
#include <mutex>

#include "common.cuh"
#include "gemm_tc.cuh"

namespace smartmem {
namespace {

template <int LPR>
__device__ __forceinline__ float group_sum(float v) {
#pragma unroll
  for (int o = LPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

__device__ __forceinline__ void unpack8_bf16(const uint4& u, float (&f)[8]) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    f[2 * q] = __uint_as_float(w[q] << 16);
    f[2 * q + 1] = __uint_as_float(w[q] & 0xFFFF0000u);
  }
}

// LPR lanes cooperate on one row and keep up to 4 16-byte vectors each in registers (vector k of
// lane l is vector l + k * LPR of the row, so a warp-wide load covers 32 / LPR rows with runs of
// LPR * 16 contiguous bytes).  RPG rows per lane group are in flight together.  GENERIC: any row
// length; the row is re-read from L1/L2 for each pass instead of being kept.
// 16-bit elements stay packed in registers (16 instead of 32 per row slice) and are unpacked for each pass: with six CTAs
// per SM the 12 544 rows of a 14 x 14 x 64 activation are all in flight in a single wave (four CTAs made it 1.3 waves).
template <typename T, int LPR, bool RMS, int RPG, bool GENERIC>
__global__ void __launch_bounds__(256, (!GENERIC && sizeof(T) == 2 && RPG == 1) ? 6 : 1) norm_kernel(const T* __restrict__ src, T* __restrict__ dst,
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
  constexpr bool PACKED = !GENERIC && sizeof(T) == 2;       // (KV == 8: one 16-byte vector)
  float v[PACKED ? 1 : RPG][PACKED ? 1 : NV][KV];
  uint4 pv[PACKED ? RPG : 1][PACKED ? NV : 1];
  auto slice = [&](int r, int k, float (&f)[KV]) {           // values of (row r, vector k) as fp32
    if constexpr (PACKED) {
      unpack8_bf16(pv[r][k], reinterpret_cast<float(&)[8]>(f));
    } else {
#pragma unroll
      for (int e = 0; e < KV; ++e) f[e] = v[r][k][e];
    }
  };
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
        if constexpr (PACKED) {
          pv[r][k] = make_uint4(0, 0, 0, 0);
          if (k < vpl && active[r] && vi < nvec) pv[r][k] = *reinterpret_cast<const uint4*>(s[r] + vi * KV);
        } else if (k < vpl && active[r] && vi < nvec) {
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
          float f[KV];
          slice(r, k, f);
#pragma unroll
          for (int e = 0; e < KV; ++e) sum[r] += RMS ? f[e] * f[e] : f[e];
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
            float f[KV];
            slice(r, k, f);
#pragma unroll
            for (int e = 0; e < KV; ++e) sq += (f[e] - mean[r]) * (f[e] - mean[r]);
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
          if (active[r]) {
            float f[KV];
            slice(r, k, f);
            emit(r, vi, f, g, b);
          }
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

// LayerNorm over a dimension that is STRIDED in the producer's buffer while the token dimension is the
// contiguous one -- a channels-first (NCHW) producer normalised over C, the implicit layout
// transformation of Fig. 1(b).  A CTA takes 64 consecutive tokens of one image.  Eight lanes cover a
// channel's 64 tokens with one 16-byte load each (128 contiguous bytes per channel), 32 channels per
// pass; a thread keeps its 8 tokens x NK channels in registers, so both statistics passes run on
// registers and only per-token partial sums cross threads (two shuffles, then shared memory across the
// eight warps).  The normalised values are written to shared memory transposed ([token][C], odd word
// pitch), from where whole channels-last rows leave with coalesced stores.  No transposed copy of the
// input is ever stored.
constexpr int NS_TOK = 64;
// 8 bf16 from global memory: one 16-byte load when the producer's strides keep it aligned, else four 4-byte loads
__device__ __forceinline__ uint4 ld_vec16(const __nv_bfloat16* p, bool aligned16) {
  if (aligned16) return *reinterpret_cast<const uint4*>(p);
  const uint32_t* q = reinterpret_cast<const uint32_t*>(p);
  return make_uint4(q[0], q[1], q[2], q[3]);
}

// Channel of slot k of a thread with channel row cr: slots come in adjacent pairs (2 cr, 2 cr + 1) + 64 (k / 2), so the
// two normalised channels of a token leave as one 32-bit shared-memory store; a pass (fixed k) still covers 32 distinct
// channel rows with eight lanes each.
__device__ __forceinline__ int ns_channel(int k, int cr) { return (k >> 1) * 64 + 2 * cr + (k & 1); }

template <int NK>                                        // channel slots per thread (even): C <= 32 * NK
__global__ void __launch_bounds__(256, NK == 8 ? 2 : 1) norm_strided_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst,
                                                           const __nv_bfloat16* __restrict__ gamma,
                                                           const __nv_bfloat16* __restrict__ beta, float eps, int C,
                                                           long long c_stride, long long img_stride, int tiles_per_img,
                                                           long long base, bool vec_ok, int n_tiles) {
  extern __shared__ __align__(16) unsigned char ns_smem[];
  const int P = C + 2;                                                      // bf16 per transposed row: (C + 2) / 2 words, odd
  __nv_bfloat16* slab = reinterpret_cast<__nv_bfloat16*>(ns_smem);          // [64][P]
  float* part = reinterpret_cast<float*>(slab + (size_t)NS_TOK * P);       // [2][8 warps][64 tokens]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tg = tid & 7, cr = tid >> 3;                                    // token group (8 tokens), channel row of a pass
  pdl_wait();
  pdl_launch_dependents();
  // persistent over the slabs: the next slab's loads are requested before this one is worked on, so every thread
  // always has NK 16-byte loads in flight
  auto request = [&](int t, uint4 (&v)[NK]) {
    const int img = t / tiles_per_img, tile = t - img * tiles_per_img;
    const __nv_bfloat16* s = src + base + (long long)img * img_stride + (long long)tile * NS_TOK + 8 * tg;
#pragma unroll
    for (int k = 0; k < NK; ++k) {
      const int c = ns_channel(k, cr);
      v[k] = make_uint4(0, 0, 0, 0);
      if (t < n_tiles && c < C) v[k] = ld_vec16(s + c * c_stride, vec_ok);
    }
  };
  uint4 r[NK], rn[NK];
  request((int)blockIdx.x, rn);
  for (int tcur = (int)blockIdx.x; tcur < n_tiles; tcur += (int)gridDim.x) {
#pragma unroll
  for (int k = 0; k < NK; ++k) r[k] = rn[k];
  request(tcur + (int)gridDim.x, rn);
  // sums of this thread's channels for its 8 tokens, then over the four channel rows of the warp, then over the warps
  auto reduce_tokens = [&](float (&v)[8], float* buf) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      v[j] += __shfl_xor_sync(0xFFFFFFFFu, v[j], 8);
      v[j] += __shfl_xor_sync(0xFFFFFFFFu, v[j], 16);
    }
    if (lane < 8) {
      float4* o = reinterpret_cast<float4*>(buf + warp * NS_TOK + 8 * tg);
      o[0] = make_float4(v[0], v[1], v[2], v[3]);
      o[1] = make_float4(v[4], v[5], v[6], v[7]);
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      const float4* i4 = reinterpret_cast<const float4*>(buf + w * NS_TOK + 8 * tg);
      const float4 a = i4[0], b = i4[1];
      v[0] += a.x; v[1] += a.y; v[2] += a.z; v[3] += a.w;
      v[4] += b.x; v[5] += b.y; v[6] += b.z; v[7] += b.w;
    }
  };
  const float invC = 1.0f / (float)C;
  float mean[8], rstd[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) mean[j] = 0.f;
#pragma unroll
  for (int k = 0; k < NK; ++k) {
    float f[8];
    unpack8_bf16(r[k], f);                                                  // absent channel slots hold zeros
#pragma unroll
    for (int j = 0; j < 8; ++j) mean[j] += f[j];
  }
  reduce_tokens(mean, part);
#pragma unroll
  for (int j = 0; j < 8; ++j) { mean[j] *= invC; rstd[j] = 0.f; }
#pragma unroll
  for (int k = 0; k < NK; ++k) {
    if (ns_channel(k, cr) < C) {
      float f[8];
      unpack8_bf16(r[k], f);
#pragma unroll
      for (int j = 0; j < 8; ++j) rstd[j] = fmaf(f[j] - mean[j], f[j] - mean[j], rstd[j]);
    }
  }
  reduce_tokens(rstd, part + 8 * NS_TOK);
#pragma unroll
  for (int j = 0; j < 8; ++j) rstd[j] = rsqrtf(rstd[j] * invC + eps);
  // normalise and store transposed: the channel pair (c, c + 1) of a token is one 32-bit word of its row (C is even)
  float ms[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) ms[j] = -mean[j] * rstd[j];
  uint32_t* slab32 = reinterpret_cast<uint32_t*>(slab);
#pragma unroll
  for (int k = 0; k < NK; k += 2) {
    const int c = ns_channel(k, cr);
    if (c < C) {
      float f0[8], f1[8];
      unpack8_bf16(r[k], f0);
      unpack8_bf16(r[k + 1], f1);
      const float2 g = bf16x2_to_float2(*reinterpret_cast<const uint32_t*>(gamma + c));
      const float2 b = bf16x2_to_float2(*reinterpret_cast<const uint32_t*>(beta + c));
#pragma unroll
      for (int j = 0; j < 8; ++j)
        slab32[(8 * tg + j) * (P / 2) + (c >> 1)] =
            float2_to_bf16x2(fmaf(fmaf(f0[j], rstd[j], ms[j]), g.x, b.x), fmaf(fmaf(f1[j], rstd[j], ms[j]), g.y, b.y));
    }
  }
  __syncthreads();
  // channels-last rows: a warp per token, a bf16 pair per lane and step
  uint32_t* d = reinterpret_cast<uint32_t*>(dst + ((long long)tcur * NS_TOK) * C);
  const uint32_t* sl = reinterpret_cast<const uint32_t*>(slab);
  for (int t = warp; t < NS_TOK; t += 8)
    for (int c2 = lane; c2 < C / 2; c2 += 32) d[(long long)t * (C / 2) + c2] = sl[t * (P / 2) + c2];
  __syncthreads();                                   // the slab is rewritten by the next round
  }
}

// The strided-channel form of a map: [images] x [tokens, contiguous] x [C, strided]; tokens a multiple of 64.
bool norm_strided_supported(const smartmem_index_map_t& m, int elem_size, long long C) {
  const int n = m.n_atoms;
  if (m.klass != 1 || elem_size != 2 || n < 2 || n > 3 || C % 2 || C > 512) return false;
  if (m.extent[n - 1] != C || m.src_stride[n - 1] == 1 || m.src_stride[n - 2] != 1 || m.extent[n - 2] % NS_TOK) return false;
  if (m.base % 2 || m.src_stride[n - 1] % 2 || (n == 3 && m.src_stride[0] % 2)) return false;
  if (m.n_elements / C / NS_TOK >= (1ll << 31)) return false;
  return true;
}

int launch_norm_strided(const void* src, void* dst, const void* gamma, const void* beta, float eps,
                        const smartmem_index_map_t& m, int C, cudaStream_t st) {
  const int n = m.n_atoms;
  const long long tokens = m.extent[n - 2], images = n == 3 ? m.extent[0] : 1;
  const size_t smem = (size_t)NS_TOK * (C + 2) * 2 + 2 * 8 * NS_TOK * sizeof(float);
  static std::mutex mu;
  static size_t configured = 48 * 1024;
  {
    std::lock_guard<std::mutex> lk(mu);
    if (smem > configured) {
      if (cudaFuncSetAttribute(norm_strided_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
          cudaFuncSetAttribute(norm_strided_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SMARTMEM_ERR_CUDA;
      configured = smem;
    }
  }
  const bool vec_ok = ((uintptr_t)src & 15) == 0 && m.base % 8 == 0 && m.src_stride[n - 1] % 8 == 0 && (n < 3 || m.src_stride[0] % 8 == 0);
  const long long n_tiles = images * (tokens / NS_TOK);
  const long long slots = (long long)tc_sm_count() * (C <= 256 ? 2 : 1);
  const dim3 grid((unsigned)(n_tiles < slots ? n_tiles : slots));
  const long long img_stride = n == 3 ? (long long)m.src_stride[0] : 0ll;
  if (C <= 256)
    launch_pdl(norm_strided_kernel<8>, grid, dim3(256), smem, st, (const __nv_bfloat16*)src, (__nv_bfloat16*)dst,
               (const __nv_bfloat16*)gamma, (const __nv_bfloat16*)beta, eps, C, (long long)m.src_stride[n - 1], img_stride,
               (int)(tokens / NS_TOK), (long long)m.base, vec_ok, (int)n_tiles);
  else
    launch_pdl(norm_strided_kernel<16>, grid, dim3(256), smem, st, (const __nv_bfloat16*)src, (__nv_bfloat16*)dst,
               (const __nv_bfloat16*)gamma, (const __nv_bfloat16*)beta, eps, C, (long long)m.src_stride[n - 1], img_stride,
               (int)(tokens / NS_TOK), (long long)m.base, vec_ok, (int)n_tiles);
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

bool layernorm_map_strided_supported(const smartmem_index_map_t& map, int elem_size, long long C) {
  return norm_strided_supported(map, elem_size, C);
}

int launch_layernorm_map(int dtype, const void* src, void* dst, const void* gamma, const void* beta, float eps,
                         const smartmem_index_map_t& map, int C, cudaStream_t st) {
  profile_tick("layernorm_map", st);
  if (dtype == SMARTMEM_BF16 && norm_strided_supported(map, 2, C)) return launch_norm_strided(src, dst, gamma, beta, eps, map, C, st);
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
