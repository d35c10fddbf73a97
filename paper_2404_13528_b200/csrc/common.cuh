// Shared device/host helpers of the CUDA path.
#pragma once
#include <cstdlib>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "smartmem.h"

namespace smartmem {

// ---------------------------------------------------------------------------------------
// Device status word (bounded waits / debug bounds) and launch accounting.
// ---------------------------------------------------------------------------------------
int* device_status_ptr();                 // device address of the status word on the CURRENT device (looked up once per device)
void count_launch(int n = 1);
// Raises a kernel's dynamic shared-memory limit, once per (device, kernel); returns a smartmem_status_t.
// `carveout` >= 0 also sets the preferred shared-memory carve-out (percent).
int ensure_max_dynamic_smem(const void* kernel, int bytes, int carveout = -1);

// Programmatic dependent launch.  A kernel launched through `launch_pdl` may start (be scheduled,
// set up its barriers and tensor memory, prefetch its descriptors and constants) while the kernel
// before it in the stream is still draining; it must call `pdl_wait()` before it reads or writes
// anything that kernel could touch.  The wait returns once the whole preceding grid has finished
// and its writes are visible.  `pdl_launch_dependents()` lets the NEXT kernel in the stream begin
// that early start as soon as every CTA of this one has called it.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// `cluster_x` > 1 launches thread-block clusters of that many CTAs (neighbours in blockIdx.x).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, unsigned cluster_x,
                                      Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  // SMARTMEM_NO_PDL=1 launches every kernel with ordinary stream ordering (for measuring what the overlap buys)
  static const int allow = [] { const char* e = getenv("SMARTMEM_NO_PDL"); return (e && e[0] == '1') ? 0 : 1; }();
  attr[0].val.programmaticStreamSerializationAllowed = allow;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cluster_x > 1) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  return launch_pdl_cluster(kernel, grid, block, smem, st, 1u, static_cast<Args&&>(args)...);
}
#endif

// When a profiling session is open (smartmem_profile_begin), records a CUDA event on `st` labelled
// `name`; every launcher calls it right before its kernel launch.
void profile_tick(const char* name, cudaStream_t st);

// ---------------------------------------------------------------------------------------
// Division by a run-time constant without a divide instruction: q = umulhi(n, mul) >> shr
// for 0 <= n < 2^31 (round-up reciprocal).  Extents are plan-time constants, so the
// reciprocals are computed once on the host.
// ---------------------------------------------------------------------------------------
struct FastDiv {
  uint32_t d, mul, shr;
};

inline FastDiv make_fastdiv(uint32_t d) {
  FastDiv f{d, 0u, 0u};
  if (d > 1) {
    uint32_t l = 0;
    while ((1ull << l) < d) ++l;        // ceil(log2 d)
    uint32_t p = 31 + l;
    f.mul = (uint32_t)(((1ull << p) + d - 1) / d);
    f.shr = p - 32;
  }
  return f;
}

__device__ __forceinline__ uint32_t fd_div(uint32_t n, const FastDiv& f) {
  return f.d == 1 ? n : (__umulhi(n, f.mul) >> f.shr);
}

// ---------------------------------------------------------------------------------------
// Device form of a canonical index map (see smartmem_index_map_t).  `unit` elements of the
// innermost atom are handled as one vector, so extent[n-1] is in vectors and offsets are
// returned in elements.
// ---------------------------------------------------------------------------------------
constexpr int kMaxDevAtoms = 10;
struct DevMap {
  int n_atoms, n_rolls;
  FastDiv ext[kMaxDevAtoms];
  long long stride[kMaxDevAtoms];       // elements; for the (vectorised) innermost atom: unit
  int roll_of[kMaxDevAtoms];
  int weight[kMaxDevAtoms];
  int roll_shift[SMARTMEM_MAX_ROLLS], roll_mod[SMARTMEM_MAX_ROLLS];
  long long roll_stride[SMARTMEM_MAX_ROLLS];
  int roll_n_parts[SMARTMEM_MAX_ROLLS];                     // > 1: decompose the wrapped coordinate again
  FastDiv roll_part_ext[SMARTMEM_MAX_ROLLS][SMARTMEM_MAX_ROLLS];
  long long roll_part_stride[SMARTMEM_MAX_ROLLS][SMARTMEM_MAX_ROLLS];
  long long base;
};

// Source offset (elements) of consumer unit `i`.  Everything stays in registers: the rolled
// coordinates are accumulated with selects instead of an indexed array.
__device__ __forceinline__ long long devmap_eval(const DevMap& m, uint32_t i) {
  long long off = m.base;
  int u0 = 0, u1 = 0, u2 = 0, u3 = 0;
#pragma unroll 1
  for (int a = m.n_atoms - 1; a >= 0; --a) {
    const uint32_t q = fd_div(i, m.ext[a]);
    const int digit = (int)(i - q * m.ext[a].d);
    i = q;
    const int r = m.roll_of[a];
    if (r < 0) {
      off += (long long)digit * m.stride[a];
    } else {
      const int w = digit * m.weight[a];
      u0 += r == 0 ? w : 0;
      u1 += r == 1 ? w : 0;
      u2 += r == 2 ? w : 0;
      u3 += r == 3 ? w : 0;
    }
  }
  auto wrap = [&](int u, int r) {
    int v = u + m.roll_shift[r];
    if (v >= m.roll_mod[r]) v -= m.roll_mod[r];     // u < mod and shift < mod: one conditional subtract
    if (m.roll_n_parts[r] <= 1) {
      off += (long long)v * m.roll_stride[r];
    } else {
      uint32_t vv = (uint32_t)v;
      for (int k = m.roll_n_parts[r] - 1; k >= 0; --k) {
        const uint32_t q = fd_div(vv, m.roll_part_ext[r][k]);
        off += (long long)(vv - q * m.roll_part_ext[r][k].d) * m.roll_part_stride[r][k];
        vv = q;
      }
    }
  };
  if (m.n_rolls > 0) wrap(u0, 0);
  if (m.n_rolls > 1) wrap(u1, 1);
  if (m.n_rolls > 2) wrap(u2, 2);
  if (m.n_rolls > 3) wrap(u3, 3);
  return off;
}

// Same result, with the atom loop fully unrolled: every map constant then is a fixed kernel-parameter
// operand of the arithmetic instead of an indexed constant load, and the digits of different atoms
// overlap (only the quotient chain is sequential).  For callers where one thread evaluates the map per
// row on a critical path; costs code size, so the copy kernels keep the rolled loop.
__device__ __forceinline__ long long devmap_eval_unrolled(const DevMap& m, uint32_t i) {
  long long off = m.base;
  int u0 = 0, u1 = 0, u2 = 0, u3 = 0;
#pragma unroll
  for (int a = kMaxDevAtoms - 1; a >= 0; --a) {
    if (a < m.n_atoms) {
      const uint32_t q = fd_div(i, m.ext[a]);
      const int digit = (int)(i - q * m.ext[a].d);
      i = q;
      const int r = m.roll_of[a];
      if (r < 0) {
        off += (long long)digit * m.stride[a];
      } else {
        const int w = digit * m.weight[a];
        u0 += r == 0 ? w : 0;
        u1 += r == 1 ? w : 0;
        u2 += r == 2 ? w : 0;
        u3 += r == 3 ? w : 0;
      }
    }
  }
#pragma unroll
  for (int r = 0; r < SMARTMEM_MAX_ROLLS; ++r) {
    if (r < m.n_rolls) {
      int v = (r == 0 ? u0 : r == 1 ? u1 : r == 2 ? u2 : u3) + m.roll_shift[r];
      if (v >= m.roll_mod[r]) v -= m.roll_mod[r];
      if (m.roll_n_parts[r] <= 1) {
        off += (long long)v * m.roll_stride[r];
      } else {
        uint32_t vv = (uint32_t)v;
#pragma unroll
        for (int k = SMARTMEM_MAX_ROLLS - 1; k >= 0; --k) {
          if (k < m.roll_n_parts[r]) {
            const uint32_t q = fd_div(vv, m.roll_part_ext[r][k]);
            off += (long long)(vv - q * m.roll_part_ext[r][k].d) * m.roll_part_stride[r][k];
            vv = q;
          }
        }
      }
    }
  }
  return off;
}

// Partial evaluation.  The digit decomposition is linear up to the final wrap of the rolled coordinates, so a consumer
// index i = n * P + t (P = the product of the extents of the trailing atoms [split, n_atoms)) can be evaluated as the sum
// of the contributions of n over the leading atoms and of t over the trailing ones, wrapped once: a kernel that walks
// over tiles (n) of P rows keeps a table of the trailing contributions and evaluates the leading atoms once per tile.
struct DevMapPart {
  long long off;
  int u0, u1, u2, u3;
};
// contribution of the digits of `i` over atoms [a0, a1) (i below the product of their extents); the base is not included
__device__ __forceinline__ DevMapPart devmap_part(const DevMap& m, int a0, int a1, uint32_t i) {
  DevMapPart p{0, 0, 0, 0, 0};
#pragma unroll
  for (int a = kMaxDevAtoms - 1; a >= 0; --a) {
    if (a >= a0 && a < a1) {
      const uint32_t q = fd_div(i, m.ext[a]);
      const int digit = (int)(i - q * m.ext[a].d);
      i = q;
      const int r = m.roll_of[a];
      if (r < 0) {
        p.off += (long long)digit * m.stride[a];
      } else {
        const int w = digit * m.weight[a];
        p.u0 += r == 0 ? w : 0;
        p.u1 += r == 1 ? w : 0;
        p.u2 += r == 2 ? w : 0;
        p.u3 += r == 3 ? w : 0;
      }
    }
  }
  return p;
}
// Same with a rolled loop over the atoms (indexed loads of the map constants): a fraction of the code, for callers that run
// once in a long while, where the fetch of the instructions costs more than their execution.
__device__ __forceinline__ DevMapPart devmap_part_rolled(const DevMap& m, int a0, int a1, uint32_t i) {
  DevMapPart p{0, 0, 0, 0, 0};
#pragma unroll 1
  for (int a = a1 - 1; a >= a0; --a) {
    const uint32_t q = fd_div(i, m.ext[a]);
    const int digit = (int)(i - q * m.ext[a].d);
    i = q;
    const int r = m.roll_of[a];
    if (r < 0) {
      p.off += (long long)digit * m.stride[a];
    } else {
      const int w = digit * m.weight[a];
      p.u0 += r == 0 ? w : 0;
      p.u1 += r == 1 ? w : 0;
      p.u2 += r == 2 ? w : 0;
      p.u3 += r == 3 ? w : 0;
    }
  }
  return p;
}
// sum of two contributions -> source offset (base added, rolled coordinates wrapped); maps with at most two rolls whose
// wrapped coordinate is an affine coordinate of the producer (roll_n_parts <= 1)
__device__ __forceinline__ long long devmap_finish2(const DevMap& m, long long off, int u0, int u1) {
  off += m.base;
  if (m.n_rolls > 0) {
    int v = u0 + m.roll_shift[0];
    if (v >= m.roll_mod[0]) v -= m.roll_mod[0];
    off += (long long)v * m.roll_stride[0];
  }
  if (m.n_rolls > 1) {
    int v = u1 + m.roll_shift[1];
    if (v >= m.roll_mod[1]) v -= m.roll_mod[1];
    off += (long long)v * m.roll_stride[1];
  }
  return off;
}
// Host: first trailing atom such that the atoms [split, n_atoms) have extents whose product is P and devmap_finish2
// applies; -1 if the map does not split there (callers then evaluate every index in full).
int devmap_split(const DevMap& m, long long P);

// Host: builds a DevMap over atoms [a0, a1) of a public map, treating `unit` elements of the
// innermost selected atom as one unit (unit must divide its extent; its stride must be 1 when
// unit > 1).  `with_base` adds the map's base.  Returns false if it does not fit.
bool make_devmap(const smartmem_index_map_t& m, int a0, int a1, int unit, bool with_base, DevMap* out);

// ---------------------------------------------------------------------------------------
// Small numeric helpers.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }
__device__ __forceinline__ float2 bf16x2_to_float2(uint32_t w) {
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
}
__device__ __forceinline__ uint32_t float2_to_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float gelu_erf(float u) { return 0.5f * u * (1.0f + erff(u * 0.70710678118654752f)); }

template <typename T> struct ElemIO;
template <> struct ElemIO<float> {
  static constexpr int kVec = 4;          // elements per 16 bytes
  __device__ static void load(const float* p, float* v) {
    float4 t = *reinterpret_cast<const float4*>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
  __device__ static void store(float* p, const float* v) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  }
  __device__ static float ld1(const float* p) { return *p; }
  __device__ static void st1(float* p, float v) { *p = v; }
};
template <> struct ElemIO<__nv_bfloat16> {
  static constexpr int kVec = 8;
  __device__ static void load(const __nv_bfloat16* p, float* v) {
    uint4 t = *reinterpret_cast<const uint4*>(p);
    float2 a = bf16x2_to_float2(t.x), b = bf16x2_to_float2(t.y), c = bf16x2_to_float2(t.z), d = bf16x2_to_float2(t.w);
    v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y; v[4] = c.x; v[5] = c.y; v[6] = d.x; v[7] = d.y;
  }
  __device__ static void store(__nv_bfloat16* p, const float* v) {
    uint4 t;
    t.x = float2_to_bf16x2(v[0], v[1]); t.y = float2_to_bf16x2(v[2], v[3]);
    t.z = float2_to_bf16x2(v[4], v[5]); t.w = float2_to_bf16x2(v[6], v[7]);
    *reinterpret_cast<uint4*>(p) = t;
  }
  __device__ static float ld1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
  __device__ static void st1(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};

// ---------------------------------------------------------------------------------------
// Launchers (defined in the .cu files).  All return a smartmem_status_t.
// ---------------------------------------------------------------------------------------
// The sequential ("no optimisation") index program of a layout run, for the device: the consumer
// index is pushed backwards through the stages with one divide/modulo chain per stage.
constexpr int kSeqMaxStages = 12, kSeqMaxDims = 8;
struct DevSeqStage {
  int kind, n_in, n_out, axis, shift;
  int in_shape[kSeqMaxDims], out_shape[kSeqMaxDims], aux[kSeqMaxDims];   // aux: perm (transpose) or start (slice)
};
struct DevSeq {
  int n_stages, n_src;
  DevSeqStage st[kSeqMaxStages];
  long long src_shape[kSeqMaxDims], src_stride[kSeqMaxDims];
};
// Copy through the sequential program (any chain; one thread per element, true div/mod).
int launch_copy_seq(const DevSeq& seq, long long n_elements, int elem_size, const void* src, void* dst, cudaStream_t st);

// Map-driven copy: out (contiguous) <- src through `map`.
// placement: 0 = best kernel for the map (tiled transposes where they apply); 1 = the plain map-driven
// gather (out[i] = src[map(i)]); 2 = the plain map-driven scatter (dst[map(i)] = src[i]).
int launch_copy_map(const smartmem_index_map_t& map, int elem_size, const void* src, void* dst, cudaStream_t st,
                    int placement = 0);

// LayerNorm / RMSNorm over rows of length C.  Row r of the output (row-major [rows, C]) is
// read from src at element offset rowmap(r) (rowmap == nullptr: r * C).
// LayerNorm over the last dimension of a [rows, C] tensor whose elements are read through `map` (consumer
// linear index -> producer element offset, 16-byte vectors intact, C / vector <= 128); writes [rows, C] contiguously.
// True when `map` is the strided-channel form (tokens contiguous in the producer, the normalised dimension strided:
// a channels-first producer) that launch_layernorm_map handles with its slab kernel.  Host only.
bool layernorm_map_strided_supported(const smartmem_index_map_t& map, int elem_size, long long C);
int launch_layernorm_map(int dtype, const void* src, void* dst, const void* gamma, const void* beta, float eps,
                         const smartmem_index_map_t& map, int C, cudaStream_t st);
int launch_norm(int dtype, bool rms, const void* src, void* dst, const void* gamma, const void* beta, float eps,
                long long rows, int C, const DevMap* rowmap, cudaStream_t st);

}  // namespace smartmem
