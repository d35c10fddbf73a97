// Causal self-attention, prefill, head dimension 128, bf16 in / fp32 softmax and accumulation.
//
// The head split ([S, 3, H, D] -> [3, H, S, D]) and the head merge ([H, S, D] -> [S, H*D]) around the
// operator are eliminated: q, k and v tiles are read as strided boxes out of the [S, 3*H*D] buffer
// the QKV GEMM wrote (rotary embedding already applied in that GEMM's epilogue), and the output
// tile is stored at column h*D of the [S, H*D] buffer the output projection reads.  The four
// strides per operand also describe the materialised [H, S, D] tensors of the explicit variant.
//
// One CTA = 64 query rows of one head (4 warps x 16 rows); keys/values stream through shared
// memory in 64-row tiles (cp.async, double buffered); scores never leave registers (online
// softmax).  Contractions use warp-level mma.sync m16n8k16.
#include <cstdlib>

#include "attn.cuh"
#include "ptx.cuh"

namespace smartmem {
namespace {

constexpr int D = 128;
constexpr int BMQ = 64, BNK = 64;
constexpr int RS = D + 8;                      // padded row, elements
constexpr int TILE_ELEMS = BNK * RS;

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ptx::smem_u32(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// 64 x 128 tile -> padded shared memory; rows >= S are zero-filled.
__device__ __forceinline__ void load_tile(__nv_bfloat16* dst, const __nv_bfloat16* src, long long st, int row0, int S,
                                          int tid) {
  for (int i = tid; i < BNK * (D / 8); i += 128) {
    const int r = i >> 4, c = i & 15;
    __nv_bfloat16* d = dst + r * RS + c * 8;
    if (row0 + r < S) cp_async16(d, src + (long long)(row0 + r) * st + c * 8);
    else *reinterpret_cast<uint4*>(d) = make_uint4(0, 0, 0, 0);
  }
}

__global__ void __launch_bounds__(128) causal_attn_kernel(const __grid_constant__ CausalAttnArgs a) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ __align__(16) __nv_bfloat16 sm[];
  __nv_bfloat16* Qs = sm;                       // [64][RS]
  __nv_bfloat16* Ks = sm + TILE_ELEMS;          // [2][64][RS]
  __nv_bfloat16* Vs = sm + 3 * TILE_ELEMS;      // [2][64][RS]

  const int n_mt = (a.S + BMQ - 1) / BMQ;
  const int mt = n_mt - 1 - (int)blockIdx.x;    // heaviest (last) query tiles first
  const int h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
  auto base = [&](const AttnOperand& o) { return (const __nv_bfloat16*)o.ptr + (long long)b * o.sn + (long long)h * o.sh; };
  const __nv_bfloat16 *qp = base(a.q), *kp = base(a.k), *vp = base(a.v);

  load_tile(Qs, qp, a.q.st, mt * BMQ, a.S, tid);
  load_tile(Ks, kp, a.k.st, 0, a.S, tid);
  load_tile(Vs, vp, a.v.st, 0, a.S, tid);
  cp_async_commit();

  constexpr int RW = RS / 2;
  uint32_t qf[8][4];
  float o[16][4];
#pragma unroll
  for (int j = 0; j < 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  const int r0 = warp * 16 + g, r1 = r0 + 8;           // rows inside the query tile
  const int qi0 = mt * BMQ + r0, qi1 = mt * BMQ + r1;   // absolute positions
  const float sl2 = a.scale * 1.4426950408889634f;      // scores are kept in the log2 domain

  const int n_nt = mt + 1;
  for (int nt = 0; nt < n_nt; ++nt) {
    const int cur = nt & 1;
    if (nt + 1 < n_nt) {
      load_tile(Ks + (cur ^ 1) * TILE_ELEMS, kp, a.k.st, (nt + 1) * BNK, a.S, tid);
      load_tile(Vs + (cur ^ 1) * TILE_ELEMS, vp, a.v.st, (nt + 1) * BNK, a.S, tid);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (nt == 0) {
      const uint32_t* Qw = reinterpret_cast<const uint32_t*>(Qs);
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        qf[kk][0] = Qw[r0 * RW + kk * 8 + t4];
        qf[kk][1] = Qw[r1 * RW + kk * 8 + t4];
        qf[kk][2] = Qw[r0 * RW + kk * 8 + 4 + t4];
        qf[kk][3] = Qw[r1 * RW + kk * 8 + 4 + t4];
      }
    }
    const uint32_t* Kw = reinterpret_cast<const uint32_t*>(Ks + cur * TILE_ELEMS);
    const __nv_bfloat16* Vt = Vs + cur * TILE_ELEMS;
    float s[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t b0 = Kw[(j * 8 + g) * RW + kk * 8 + t4];
        const uint32_t b1 = Kw[(j * 8 + g) * RW + kk * 8 + 4 + t4];
        ptx::mma_m16n8k16_bf16(s[j], qf[kk], b0, b1);
      }
    }
    // scale, causal mask (only the diagonal tile needs it), online softmax
    const bool diag = (nt == mt);
    float mx0 = m0, mx1 = m1;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int kj = nt * BNK + j * 8 + 2 * t4 + e;
        float v0 = s[j][e] * sl2, v1 = s[j][2 + e] * sl2;
        if (diag) {
          if (kj > qi0) v0 = -INFINITY;
          if (kj > qi1) v1 = -INFINITY;
        }
        s[j][e] = v0;
        s[j][2 + e] = v1;
        mx0 = fmaxf(mx0, v0);
        mx1 = fmaxf(mx1, v1);
      }
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 2));
    const float c0 = exp2f(m0 - mx0), c1 = exp2f(m1 - mx1);     // first tile: exp2(-inf) = 0
    m0 = mx0;
    m1 = mx1;
    float rs0 = 0.f, rs1 = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const float p0 = exp2f(s[j][e] - m0), p1 = exp2f(s[j][2 + e] - m1);
        s[j][e] = p0;
        s[j][2 + e] = p1;
        rs0 += p0;
        rs1 += p1;
      }
    }
    l0 = l0 * c0 + rs0;
    l1 = l1 * c1 + rs1;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      o[j][0] *= c0; o[j][1] *= c0; o[j][2] *= c1; o[j][3] *= c1;
    }
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      uint32_t af[4];
      af[0] = float2_to_bf16x2(s[2 * kk][0], s[2 * kk][1]);
      af[1] = float2_to_bf16x2(s[2 * kk][2], s[2 * kk][3]);
      af[2] = float2_to_bf16x2(s[2 * kk + 1][0], s[2 * kk + 1][1]);
      af[3] = float2_to_bf16x2(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        uint32_t b0, b1;
        const __nv_bfloat16* rowp = Vt + (kk * 16 + (lane & 15)) * RS + j * 8;
        asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];"
                     : "=r"(b0), "=r"(b1)
                     : "r"(ptx::smem_u32(rowp)));
        ptx::mma_m16n8k16_bf16(o[j], af, b0, b1);
      }
    }
    __syncthreads();                             // the other buffer is refilled next iteration
  }
  l0 += __shfl_xor_sync(0xFFFFFFFFu, l0, 1);
  l0 += __shfl_xor_sync(0xFFFFFFFFu, l0, 2);
  l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, 1);
  l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, 2);
  const float i0 = 1.f / l0, i1 = 1.f / l1;
  __nv_bfloat16* op = (__nv_bfloat16*)a.o.ptr + (long long)b * a.o.sn + (long long)h * a.o.sh;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const int c = j * 8 + 2 * t4;
    if (qi0 < a.S) *reinterpret_cast<uint32_t*>(op + (long long)qi0 * a.o.st + c) = float2_to_bf16x2(o[j][0] * i0, o[j][1] * i0);
    if (qi1 < a.S) *reinterpret_cast<uint32_t*>(op + (long long)qi1 * a.o.st + c) = float2_to_bf16x2(o[j][2] * i1, o[j][3] * i1);
  }
}

// cos/sin table of the rotary embedding: tab[p, i] = (cos, sin)(p * theta^(-2i/D)), i < D/2.
__global__ void rope_table_kernel(float2* tab, int S, int half, double theta) {
  pdl_wait();
  pdl_launch_dependents();
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= S * half) return;
  const int p = idx / half, i = idx - p * half;
  const double ang = (double)p * pow(theta, -(double)i / (double)half);
  tab[idx] = make_float2((float)cos(ang), (float)sin(ang));
}

// Stand-alone rotary embedding (explicit variant): rows of [R, D] with position = row % S.
__global__ void rope_rows_kernel(__nv_bfloat16* x, long long rows, int S, int Dh, int rot, const float2* __restrict__ tab) {
  pdl_wait();
  pdl_launch_dependents();
  const int half = rot / 2;                     // pairs (i, i + rot/2) of the first rot elements of a row of Dh
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * half) return;
  const long long r = idx / half;
  const int i = (int)(idx - r * half);
  const float2 cs = tab[(r % S) * half + i];
  __nv_bfloat16* row = x + r * Dh;
  const float a = __bfloat162float(row[i]), b = __bfloat162float(row[i + half]);
  row[i] = __float2bfloat16_rn(a * cs.x - b * cs.y);
  row[i + half] = __float2bfloat16_rn(b * cs.x + a * cs.y);
}

}  // namespace

int launch_causal_attention_tc(const CausalAttnArgs& a, cudaStream_t st);

int launch_causal_attention(const CausalAttnArgs& a, cudaStream_t st) {
  // tcgen05 path for the two operand layouts it knows; SMARTMEM_CAUSAL_LEGACY=1 keeps the warp-MMA kernel
  static const bool legacy = [] { const char* e = getenv("SMARTMEM_CAUSAL_LEGACY"); return e && e[0] == '1'; }();
  if (!legacy) {
    const int rc = launch_causal_attention_tc(a, st);
    if (rc != SMARTMEM_ERR_UNSUPPORTED) return rc;
  }
  if (a.S < 1 || a.heads < 1 || a.batch < 1 || a.heads > 65535 || a.batch > 65535) return SMARTMEM_ERR_UNSUPPORTED;
  const AttnOperand* ops[4] = {&a.q, &a.k, &a.v, &a.o};
  for (auto* o : ops)
    if (o->se != 1 || o->st % 8 || o->sn % 8 || o->sh % 8 || ((uintptr_t)o->ptr & 15)) return SMARTMEM_ERR_ALIGNMENT;
  const size_t smem = 5 * (size_t)TILE_ELEMS * 2;
  if (ensure_max_dynamic_smem((const void*)causal_attn_kernel, (int)smem) != SMARTMEM_OK) return SMARTMEM_ERR_CUDA;
  profile_tick("causal_attention", st);
  dim3 grid((a.S + BMQ - 1) / BMQ, a.heads, a.batch);
  launch_pdl(causal_attn_kernel, dim3(grid), dim3(128), smem, st, a);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

int launch_rope_table(float* tab, int S, int head_dim, float theta, cudaStream_t st) {
  const int n = S * (head_dim / 2);
  profile_tick("rope_table", st);
  launch_pdl(rope_table_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, (float2*)tab, S, head_dim / 2, (double)theta);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

int launch_rope_rows(void* x, long long rows, int S, int head_dim, const float* tab, cudaStream_t st, int rotary_dim) {
  const int rot = rotary_dim ? rotary_dim : head_dim;
  const long long n = rows * (rot / 2);
  profile_tick("rope_rows", st);
  launch_pdl(rope_rows_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, (__nv_bfloat16*)x, rows, S, head_dim, rot, (const float2*)tab);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

}  // namespace smartmem
