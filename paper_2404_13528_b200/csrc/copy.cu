// Map-driven copy kernels: the consumer is the identity, so the kernel is exactly the
// composed index map of an eliminated layout run (Section 3.2.1) applied on the load side.
// They serve the copy-only chains and every materialised layout operator of EXPLICIT mode.
#include <vector>

#include "common.cuh"

namespace smartmem {

bool make_devmap(const smartmem_index_map_t& m, int a0, int a1, int unit, bool with_base, DevMap* out) {
  if (a1 - a0 > kMaxDevAtoms || a0 < 0 || a1 > m.n_atoms) return false;
  DevMap d;
  memset(&d, 0, sizeof(d));
  d.n_atoms = a1 - a0;
  d.n_rolls = m.n_rolls;
  d.base = with_base ? m.base : 0;
  for (int r = 0; r < m.n_rolls; ++r) {
    if (m.roll_mod[r] >= (1ll << 30)) return false;
    d.roll_shift[r] = (int)m.roll_shift[r];
    d.roll_mod[r] = (int)m.roll_mod[r];
    d.roll_stride[r] = m.roll_stride[r];
    d.roll_n_parts[r] = m.roll_n_parts[r];
    for (int k = 0; k < m.roll_n_parts[r] && k < SMARTMEM_MAX_ROLLS; ++k) {
      if (m.roll_part_extent[r][k] >= (1ll << 31)) return false;
      d.roll_part_ext[r][k] = make_fastdiv((uint32_t)m.roll_part_extent[r][k]);
      d.roll_part_stride[r][k] = m.roll_part_stride[r][k];
    }
  }
  for (int a = a0; a < a1; ++a) {
    int64_t e = m.extent[a];
    long long s = m.src_stride[a];
    if (a == a1 - 1 && unit > 1) {
      if (m.roll_of[a] >= 0 || s != 1 || e % unit) return false;
      e /= unit;
      s = unit;
    }
    if (e >= (1ll << 31) || m.roll_weight[a] >= (1ll << 30)) return false;
    d.ext[a - a0] = make_fastdiv((uint32_t)e);
    d.stride[a - a0] = s;
    d.roll_of[a - a0] = m.roll_of[a];
    d.weight[a - a0] = (int)m.roll_weight[a];
  }
  *out = d;
  return true;
}

int devmap_split(const DevMap& m, long long P) {
  if (m.n_rolls > 2) return -1;
  for (int r = 0; r < m.n_rolls; ++r)
    if (m.roll_n_parts[r] > 1) return -1;
  long long prod = 1;
  int a = m.n_atoms;
  while (a > 0 && prod < P) prod *= m.ext[--a].d;
  return prod == P ? a : -1;
}

namespace {

template <int VB> struct VecT;
template <> struct VecT<16> { using type = uint4; };
template <> struct VecT<8> { using type = uint2; };
template <> struct VecT<4> { using type = uint32_t; };
template <> struct VecT<2> { using type = uint16_t; };

// One thread per output vector of VB bytes: decompose the vector index over the atoms,
// load through the map, store contiguously (coalesced).
template <int VB>
__global__ void __launch_bounds__(256) copy_gather_kernel(const __grid_constant__ DevMap map, const char* __restrict__ src,
                                                          char* __restrict__ dst, uint32_t n_units, int elem_size) {
  pdl_wait();
  pdl_launch_dependents();
  using V = typename VecT<VB>::type;
  uint32_t i = blockIdx.x * 256u + threadIdx.x;
  if (i >= n_units) return;
  long long off = devmap_eval_unrolled(map, i);
  V v = *reinterpret_cast<const V*>(src + off * elem_size);
  *reinterpret_cast<V*>(dst + (size_t)i * VB) = v;
}

// The same map placed on the producer side: one thread per INPUT vector, loaded contiguously
// (coalesced) and stored through the map (here the map of the inverted chain: where each input
// vector goes).  The sub-optimal access is the write instead of the read.
template <int VB>
__global__ void __launch_bounds__(256) copy_scatter_kernel(const __grid_constant__ DevMap map, const char* __restrict__ src,
                                                           char* __restrict__ dst, uint32_t n_units, int elem_size) {
  pdl_wait();
  pdl_launch_dependents();
  using V = typename VecT<VB>::type;
  uint32_t i = blockIdx.x * 256u + threadIdx.x;
  if (i >= n_units) return;
  long long off = devmap_eval_unrolled(map, i);
  V v = *reinterpret_cast<const V*>(src + (size_t)i * VB);
  *reinterpret_cast<V*>(dst + off * elem_size) = v;
}

// Affine map whose innermost consumer atom is SHORT (E <= 8 values, strided in the source) and whose next
// atom is contiguous in the source -- the interleave of DepthToSpace / pixel shuffle, where neighbouring
// output elements come from E different planes.  A thread loads one 16-byte vector from each of the E
// planes (8 consecutive positions of the contiguous atom), interleaves them in registers and stores
// 8 * E contiguous output elements: both sides move 16-byte vectors, nothing goes through shared memory.
template <int E>
__global__ void __launch_bounds__(256) copy_interleave16_kernel(const __grid_constant__ DevMap map, const uint16_t* __restrict__ src,
                                                                uint16_t* __restrict__ dst, uint32_t n_units, long long stride_e) {
  pdl_wait();
  pdl_launch_dependents();
  const uint32_t i = blockIdx.x * 256u + threadIdx.x;
  if (i >= n_units) return;
  const long long off = devmap_eval_unrolled(map, i);
  uint32_t w[E][4];
#pragma unroll
  for (int j = 0; j < E; ++j) {
    const uint4 v = *reinterpret_cast<const uint4*>(src + off + j * stride_e);
    w[j][0] = v.x; w[j][1] = v.y; w[j][2] = v.z; w[j][3] = v.w;
  }
  uint32_t o[4 * E];
#pragma unroll
  for (int m = 0; m < 4 * E; ++m) {
    // output elements 2m and 2m+1: element t = k * E + j is position k of plane j
    const int k0 = (2 * m) / E, j0 = (2 * m) % E, k1 = (2 * m + 1) / E, j1 = (2 * m + 1) % E;
    const uint32_t sel = ((k0 & 1) ? 0x32u : 0x10u) | (((k1 & 1) ? 0x76u : 0x54u) << 8);
    o[m] = __byte_perm(w[j0][k0 >> 1], w[j1][k1 >> 1], sel);
  }
  uint4* d = reinterpret_cast<uint4*>(dst + (size_t)i * (8 * E));
#pragma unroll
  for (int j = 0; j < E; ++j) d[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
}

// Affine map whose consumer-innermost atom I is strided in the source while another atom J is
// source-contiguous: a 64 x 64 tile transpose of 2-byte elements through shared memory.  Loads are
// 16-byte vectors along J, stores 16-byte vectors along I.
struct TransposeArgs {
  int n_outer;
  FastDiv outer_ext[kMaxDevAtoms];
  long long outer_src[kMaxDevAtoms], outer_dst[kMaxDevAtoms];
  long long src_stride_i, dst_stride_j, base;
  int tiles_i, tiles_j;
};

__global__ void __launch_bounds__(256) copy_transpose16_kernel(const __grid_constant__ TransposeArgs a,
                                                               const uint16_t* __restrict__ src, uint16_t* __restrict__ dst) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ uint32_t tile[64][33];          // [j][i-pair]
  uint32_t b = blockIdx.x;
  uint32_t tj = b % a.tiles_j;
  b /= a.tiles_j;
  uint32_t ti = b % a.tiles_i;
  b /= a.tiles_i;
  long long so = a.base, dof = 0;
  for (int k = a.n_outer - 1; k >= 0; --k) {
    uint32_t q = fd_div(b, a.outer_ext[k]);
    uint32_t digit = b - q * a.outer_ext[k].d;
    b = q;
    so += (long long)digit * a.outer_src[k];
    dof += (long long)digit * a.outer_dst[k];
  }
  const int tid = threadIdx.x;
  {
    const int p = tid >> 3, jg = tid & 7;
    const uint16_t* s0 = src + so + (long long)(ti * 64 + 2 * p) * a.src_stride_i + tj * 64 + jg * 8;
    uint4 r0 = *reinterpret_cast<const uint4*>(s0);
    uint4 r1 = *reinterpret_cast<const uint4*>(s0 + a.src_stride_i);
    const uint32_t w0[4] = {r0.x, r0.y, r0.z, r0.w}, w1[4] = {r1.x, r1.y, r1.z, r1.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      tile[jg * 8 + 2 * e][p] = (w0[e] & 0xFFFFu) | (w1[e] << 16);
      tile[jg * 8 + 2 * e + 1][p] = (w0[e] >> 16) | (w1[e] & 0xFFFF0000u);
    }
  }
  __syncthreads();
#pragma unroll
  for (int pass = 0; pass < 2; ++pass) {
    const int q = tid & 7, j = (tid >> 3) + 32 * pass;
    uint4 v;
    v.x = tile[j][4 * q + 0];
    v.y = tile[j][4 * q + 1];
    v.z = tile[j][4 * q + 2];
    v.w = tile[j][4 * q + 3];
    *reinterpret_cast<uint4*>(dst + dof + (long long)(tj * 64 + j) * a.dst_stride_j + ti * 64 + q * 8) = v;
  }
}


// Batched transpose of small contiguous blocks: the last two consumer atoms are (J, I) of a
// source block [I][J] that is contiguous (stride of I == extent of J), e.g. a materialised K^T of
// one (window, head).  One CTA per block: coalesced 16-byte loads of the whole block into shared
// memory, coalesced 4-byte stores of the transposed block.
__global__ void __launch_bounds__(256) copy_block_transpose16_kernel(const __grid_constant__ DevMap outer,
                                                                     const uint16_t* __restrict__ src,
                                                                     uint16_t* __restrict__ dst, int EI, int EJ) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ uint16_t blk[];
  const int RS = EJ + 2;
  const int E = EI * EJ;
  const long long so = devmap_eval(outer, blockIdx.x);
  const uint16_t* sp = src + so;
  uint16_t* dp = dst + (long long)blockIdx.x * E;
  if ((so & 7) == 0 && (EJ & 7) == 0) {
    for (int l = threadIdx.x * 8; l < E; l += 256 * 8) {
      const uint4 v = *reinterpret_cast<const uint4*>(sp + l);
      const int i = l / EJ, j = l - i * EJ;
      uint32_t* d32 = reinterpret_cast<uint32_t*>(blk + i * RS + j);
      d32[0] = v.x; d32[1] = v.y; d32[2] = v.z; d32[3] = v.w;
    }
  } else {
    for (int l = threadIdx.x; l < E; l += 256) {
      const int i = l / EJ, j = l - i * EJ;
      blk[i * RS + j] = sp[l];
    }
  }
  __syncthreads();
  for (int q = threadIdx.x * 2; q < E; q += 512) {        // E is even (checked by the launcher)
    int j0 = q / EI, i0 = q - j0 * EI;
    int i1 = i0 + 1, j1 = j0;
    if (i1 == EI) { i1 = 0; ++j1; }
    const uint32_t v = (uint32_t)blk[i0 * RS + j0] | ((uint32_t)blk[i1 * RS + j1] << 16);
    *reinterpret_cast<uint32_t*>(dp + q) = v;
  }
}

// The unoptimised form of an eliminated run (Fig. 4, right): every stage delinearises the index
// in its output shape and linearises it in its input shape with run-time divides and modulos.
template <typename E>
__global__ void __launch_bounds__(256) copy_seq_kernel(const __grid_constant__ DevSeq q, const E* __restrict__ src,
                                                       E* __restrict__ dst, long long n) {
  pdl_wait();
  pdl_launch_dependents();
  const long long i0 = (long long)blockIdx.x * 256 + threadIdx.x;
  if (i0 >= n) return;
  long long idx = i0;
  for (int si = q.n_stages - 1; si >= 0; --si) {
    const DevSeqStage& st = q.st[si];
    long long c[kSeqMaxDims], in[kSeqMaxDims];
    for (int k = st.n_out - 1; k >= 0; --k) {
      c[k] = idx % st.out_shape[k];
      idx /= st.out_shape[k];
    }
    if (st.kind == SMARTMEM_OP_RESHAPE) {
      long long lin = 0;
      for (int k = 0; k < st.n_out; ++k) lin = lin * st.out_shape[k] + c[k];
      idx = lin;
      continue;
    }
    for (int k = 0; k < st.n_in; ++k) in[k] = 0;
    if (st.kind == SMARTMEM_OP_TRANSPOSE) {
      for (int k = 0; k < st.n_out; ++k) in[st.aux[k]] = c[k];
    } else if (st.kind == SMARTMEM_OP_ROLL) {
      for (int k = 0; k < st.n_out; ++k) in[k] = c[k];
      long long v = (c[st.axis] - st.shift) % st.in_shape[st.axis];
      in[st.axis] = v < 0 ? v + st.in_shape[st.axis] : v;
    } else {                                      // slice
      for (int k = 0; k < st.n_out; ++k) in[k] = c[k] + st.aux[k];
    }
    long long lin = 0;
    for (int k = 0; k < st.n_in; ++k) lin = lin * st.in_shape[k] + in[k];
    idx = lin;
  }
  long long off = 0;
  for (int k = q.n_src - 1; k >= 0; --k) {
    off += (idx % q.src_shape[k]) * q.src_stride[k];
    idx /= q.src_shape[k];
  }
  dst[i0] = src[off];
}

}  // namespace

int launch_copy_seq(const DevSeq& seq, long long n, int elem_size, const void* src, void* dst, cudaStream_t st) {
  profile_tick("copy_seq", st);
  if (n == 0) return SMARTMEM_OK;
  const long long blocks = (n + 255) / 256;
  if (blocks >= (1ll << 31)) return SMARTMEM_ERR_UNSUPPORTED;
  if (elem_size == 2) launch_pdl(copy_seq_kernel<uint16_t>, dim3((unsigned)blocks), dim3(256), 0, st, seq, (const uint16_t*)src, (uint16_t*)dst, n);
  else if (elem_size == 4) launch_pdl(copy_seq_kernel<uint32_t>, dim3((unsigned)blocks), dim3(256), 0, st, seq, (const uint32_t*)src, (uint32_t*)dst, n);
  else return SMARTMEM_ERR_UNSUPPORTED;
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

int launch_copy_map(const smartmem_index_map_t& map, int elem_size, const void* src, void* dst, cudaStream_t st, int placement) {
  profile_tick(placement == 2 ? "copy_map_scatter" : placement == 1 ? "copy_map_gather" : "copy_map", st);
  if (map.klass == 3) return SMARTMEM_ERR_UNSUPPORTED;
  if (map.n_elements == 0) return SMARTMEM_OK;
  const int n = map.n_atoms;
  if (placement == 0) {
  // fast path: batched transpose of small contiguous blocks
  if (map.klass == 1 && elem_size == 2 && n >= 2 && map.src_stride[n - 1] != 1 && map.src_stride[n - 2] == 1 &&
      map.src_stride[n - 1] == map.extent[n - 2] && map.extent[n - 1] * map.extent[n - 2] <= 16384 &&
      (map.extent[n - 1] * map.extent[n - 2]) % 2 == 0) {
    DevMap outer;
    long long blocks = map.n_elements / (map.extent[n - 1] * map.extent[n - 2]);
    if (make_devmap(map, 0, n - 2, 1, true, &outer) && blocks < (1ll << 31)) {
      const int EI = (int)map.extent[n - 1], EJ = (int)map.extent[n - 2];
      const size_t smem = (size_t)EI * (EJ + 2) * 2;
      if (smem <= 40000) {
      launch_pdl(copy_block_transpose16_kernel, dim3((unsigned)blocks), dim3(256), smem, st, outer, (const uint16_t*)src, (uint16_t*)dst, EI, EJ);
      count_launch();
      return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
      }
    }
  }
  // fast path: short strided innermost atom over a contiguous one (register interleave)
  if (map.klass == 1 && elem_size == 2 && n >= 2 && map.src_stride[n - 1] != 1 && map.src_stride[n - 2] == 1 &&
      map.extent[n - 1] >= 2 && map.extent[n - 1] <= 4 && map.extent[n - 2] % 8 == 0 && map.base % 8 == 0 &&
      map.src_stride[n - 1] % 8 == 0) {
    bool ok = true;
    for (int a = 0; a + 2 < n; ++a) ok = ok && map.src_stride[a] % 8 == 0;
    const int E = (int)map.extent[n - 1];
    const long long units = map.n_elements / (8 * E);
    DevMap d;
    if (ok && units < (1ll << 31) && make_devmap(map, 0, n - 1, 8, true, &d)) {
      const unsigned grid = (unsigned)((units + 255) / 256);
      const uint16_t* s16 = (const uint16_t*)src;
      uint16_t* d16 = (uint16_t*)dst;
      if (E == 2) launch_pdl(copy_interleave16_kernel<2>, dim3(grid), dim3(256), 0, st, d, s16, d16, (uint32_t)units, map.src_stride[n - 1]);
      else if (E == 3) launch_pdl(copy_interleave16_kernel<3>, dim3(grid), dim3(256), 0, st, d, s16, d16, (uint32_t)units, map.src_stride[n - 1]);
      else launch_pdl(copy_interleave16_kernel<4>, dim3(grid), dim3(256), 0, st, d, s16, d16, (uint32_t)units, map.src_stride[n - 1]);
      count_launch();
      return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
    }
  }
  // fast path: tiled transpose
  if (map.klass == 1 && elem_size == 2 && n >= 2 && map.src_stride[n - 1] != 1) {
    int J = -1;
    for (int a = 0; a < n - 1; ++a)
      if (map.src_stride[a] == 1) J = a;
    if (J >= 0 && map.extent[n - 1] % 64 == 0 && map.extent[J] % 64 == 0 && n - 2 <= kMaxDevAtoms) {
      TransposeArgs t;
      memset(&t, 0, sizeof(t));
      std::vector<long long> cstride(n);
      long long run = 1;
      for (int a = n - 1; a >= 0; --a) {
        cstride[a] = run;
        run *= map.extent[a];
      }
      bool ok = map.base % 8 == 0 && map.src_stride[n - 1] % 8 == 0 && cstride[J] % 8 == 0;
      long long outer = 1;
      for (int a = 0; a < n - 1; ++a) {
        if (a == J) continue;
        ok = ok && map.src_stride[a] % 8 == 0 && cstride[a] % 8 == 0 && map.extent[a] < (1ll << 31);
        t.outer_ext[t.n_outer] = make_fastdiv((uint32_t)map.extent[a]);
        t.outer_src[t.n_outer] = map.src_stride[a];
        t.outer_dst[t.n_outer] = cstride[a];
        ++t.n_outer;
        outer *= map.extent[a];
      }
      t.src_stride_i = map.src_stride[n - 1];
      t.dst_stride_j = cstride[J];
      t.base = map.base;
      t.tiles_i = (int)(map.extent[n - 1] / 64);
      t.tiles_j = (int)(map.extent[J] / 64);
      long long blocks = outer * t.tiles_i * t.tiles_j;
      if (ok && blocks < (1ll << 31)) {
        launch_pdl(copy_transpose16_kernel, dim3((unsigned)blocks), dim3(256), 0, st, t, (const uint16_t*)src, (uint16_t*)dst);
        count_launch();
        return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
      }
    }
  }
  }   // placement == 0: the tiled fast paths above; 1 / 2: the plain map-driven kernel on the consumer / producer side
  const int v = map.vec_elems;
  const int vb = v * elem_size;
  DevMap d;
  if (!make_devmap(map, 0, n, v, true, &d)) return SMARTMEM_ERR_UNSUPPORTED;
  long long units = map.n_elements / v;
  if (units >= (1ll << 31)) return SMARTMEM_ERR_UNSUPPORTED;
  unsigned grid = (unsigned)((units + 255) / 256);
#define SM_COPY(VB_)                                                                                                     \
  case VB_:                                                                                                              \
    if (placement == 2)                                                                                                  \
      launch_pdl(copy_scatter_kernel<VB_>, dim3(grid), dim3(256), 0, st, d, (const char*)src, (char*)dst, (uint32_t)units, elem_size); \
    else                                                                                                                 \
      launch_pdl(copy_gather_kernel<VB_>, dim3(grid), dim3(256), 0, st, d, (const char*)src, (char*)dst, (uint32_t)units, elem_size);  \
    break;
  switch (vb) {
    SM_COPY(16) SM_COPY(8) SM_COPY(4) SM_COPY(2)
    default: return SMARTMEM_ERR_UNSUPPORTED;
  }
#undef SM_COPY
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

}  // namespace smartmem
