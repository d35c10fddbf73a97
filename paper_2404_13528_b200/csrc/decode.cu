// smartmem_attn_decode: one decode step of the decoder attention layer against a key/value cache.
//
// ELIMINATE: RMSNorm -> fused QKV GEMM whose epilogue rotates the q and k columns at position `pos`
// and stores the k and v columns of sequence b straight into row (b, pos) of the token-major caches
// [B, S_max, heads, D] (the Concat is the producer's store) -> decode attention reading head h of the
// cache as a strided slice (head split eliminated) and writing column h*D of [B, hidden] (head merge
// eliminated) -> output projection (+ residual).  No copy kernel.
// EXPLICIT: plain QKV GEMM, head-split copy to [3, B, heads, 1, D], stand-alone rotary pass, append copy
// into the per-head caches [B, heads, S_max, D], the same attention kernel on contiguous per-head
// tensors, output projection.
//
// The attention kernel is bandwidth work: every cached key and value is read once (2 * 256 bytes per
// position and head) and used for one 128-long dot product or one 128-wide axpy, so it runs on the
// ordinary FMA pipe with 16-byte loads; the tensor cores would multiply a one-row query tile.
#include <cuda_bf16.h>

#include <map>
#include <mutex>
#include <tuple>

#include "attn.cuh"
#include "chain_util.hpp"
#include "common.cuh"
#include "gemm_tc.cuh"

#define EXPORT extern "C" __attribute__((visibility("default")))

using namespace smartmem;

namespace {

constexpr int DH = 128;                  // head dimension
constexpr int DEC_THREADS = 256;         // 8 warps = 16 half-warps, one cached position per half-warp per step
constexpr int DEC_GROUPS = DEC_THREADS / 16;
constexpr int DEC_UNROLL = 4;            // 16-byte loads in flight per thread
constexpr int DEC_MAX_S = 16384;         // scores of one (sequence, head) are kept in shared memory

struct DecodeAttnArgs {
  const __nv_bfloat16* q;  long long q_sb, q_sh;          // q[b, h, :] = q + b*q_sb + h*q_sh
  const __nv_bfloat16* k;  const __nv_bfloat16* v;
  long long kv_sb, kv_sh, kv_ss;                          // cache[b, h, s, :] = base + b*kv_sb + h*kv_sh + s*kv_ss
  __nv_bfloat16* o;        long long o_sb, o_sh;
  int heads, S;                                           // S = positions attended (cached + the new one)
  float scale_log2e;                                      // head_dim^-1/2 * log2(e)
};

__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8]) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    f[2 * j] = __uint_as_float(w[j] << 16);
    f[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
  }
}

// One CTA per (sequence, head).  Sixteen lanes share a cached row (16 bytes each); pass 1 leaves
// the scaled scores in shared memory, pass 2 accumulates exp2(score - max) * v with each lane owning 8
// of the 128 output columns, and the sixteen partial sums are added through shared memory.
__global__ void __launch_bounds__(DEC_THREADS) decode_attn_kernel(const DecodeAttnArgs a) {
  extern __shared__ float dsm[];
  float* sc = dsm;                                    // [S] scores, then probabilities
  float* part = dsm + ((a.S + 3) & ~3);               // [DEC_GROUPS][128] partial outputs
  __shared__ float red[DEC_THREADS / 32];
  __shared__ float bcast[2];
  pdl_wait();
  pdl_launch_dependents();
  const int b = blockIdx.x / a.heads, h = blockIdx.x - b * a.heads;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int l16 = tid & 15, grp = tid >> 4;
  const __nv_bfloat16* kb = a.k + b * a.kv_sb + h * a.kv_sh + l16 * 8;
  const __nv_bfloat16* vb = a.v + b * a.kv_sb + h * a.kv_sh + l16 * 8;
  float qf[8];
  unpack8(*reinterpret_cast<const uint4*>(a.q + b * a.q_sb + h * a.q_sh + l16 * 8), qf);
#pragma unroll
  for (int j = 0; j < 8; ++j) qf[j] *= a.scale_log2e;

  // ---- pass 1: scores (already in the exp2 domain) and their maximum
  float mx = -INFINITY;
  for (int base = 0; base < a.S; base += DEC_GROUPS * DEC_UNROLL) {   // trip count uniform over the CTA (shuffles below)
    const int s0 = base + grp;
    uint4 kv[DEC_UNROLL];
#pragma unroll
    for (int u = 0; u < DEC_UNROLL; ++u) {
      const int s = s0 + u * DEC_GROUPS;
      kv[u] = make_uint4(0, 0, 0, 0);
      if (s < a.S) kv[u] = __ldg(reinterpret_cast<const uint4*>(kb + s * a.kv_ss));
    }
#pragma unroll
    for (int u = 0; u < DEC_UNROLL; ++u) {
      const int s = s0 + u * DEC_GROUPS;
      float kf[8];
      unpack8(kv[u], kf);
      float d0 = 0.f, d1 = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        d0 = fmaf(qf[2 * j], kf[2 * j], d0);
        d1 = fmaf(qf[2 * j + 1], kf[2 * j + 1], d1);
      }
      float d = d0 + d1;
#pragma unroll
      for (int m = 8; m >= 1; m >>= 1) d += __shfl_xor_sync(0xFFFFFFFFu, d, m);
      if (s < a.S) {
        mx = fmaxf(mx, d);
        if (l16 == 0) sc[s] = d;
      }
    }
  }
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, m));
  if (lane == 0) red[warp] = mx;
  __syncthreads();
  if (tid == 0) {
    float m = red[0];
#pragma unroll
    for (int w = 1; w < DEC_THREADS / 32; ++w) m = fmaxf(m, red[w]);
    bcast[0] = m;
  }
  __syncthreads();
  mx = bcast[0];

  // ---- probabilities (unnormalised) and their sum
  float sum = 0.f;
  for (int s = tid; s < a.S; s += DEC_THREADS) {
    const float p = exp2f(sc[s] - mx);
    sc[s] = p;
    sum += p;
  }
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, m);
  if (lane == 0) red[warp] = sum;
  __syncthreads();
  if (tid == 0) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < DEC_THREADS / 32; ++w) t += red[w];
    bcast[1] = 1.0f / t;
  }

  // ---- pass 2: sum_s p[s] * v[s, :]
  float acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.f;
  for (int base = 0; base < a.S; base += DEC_GROUPS * DEC_UNROLL) {
    const int s0 = base + grp;
    uint4 vv[DEC_UNROLL];
    float pp[DEC_UNROLL];
#pragma unroll
    for (int u = 0; u < DEC_UNROLL; ++u) {
      const int s = s0 + u * DEC_GROUPS;
      vv[u] = make_uint4(0, 0, 0, 0);
      pp[u] = 0.f;
      if (s < a.S) {
        vv[u] = __ldg(reinterpret_cast<const uint4*>(vb + s * a.kv_ss));
        pp[u] = sc[s];
      }
    }
#pragma unroll
    for (int u = 0; u < DEC_UNROLL; ++u) {
      float vf[8];
      unpack8(vv[u], vf);
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] = fmaf(pp[u], vf[j], acc[j]);
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) part[grp * DH + l16 * 8 + j] = acc[j];
  __syncthreads();
  if (tid < DH) {
    float t = 0.f;
#pragma unroll
    for (int g = 0; g < DEC_GROUPS; ++g) t += part[g * DH + tid];
    a.o[b * a.o_sb + h * a.o_sh + tid] = __float2bfloat16_rn(t * bcast[1]);
  }
}

int launch_decode_attention(const DecodeAttnArgs& a, int B, cudaStream_t st) {
  if (a.S < 1 || a.S > DEC_MAX_S || B < 1 || a.heads < 1) return SMARTMEM_ERR_UNSUPPORTED;
  if ((long long)B * a.heads >= (1ll << 31)) return SMARTMEM_ERR_UNSUPPORTED;
  const long long strides[] = {a.q_sb, a.q_sh, a.kv_sb, a.kv_sh, a.kv_ss, a.o_sb, a.o_sh};
  for (long long s : strides)
    if (s % 8) return SMARTMEM_ERR_ALIGNMENT;
  const void* ptrs[] = {a.q, a.k, a.v, a.o};
  for (const void* p : ptrs)
    if ((uintptr_t)p & 15) return SMARTMEM_ERR_ALIGNMENT;
  const size_t smem = ((size_t)((a.S + 3) & ~3) + DEC_GROUPS * DH) * sizeof(float);
  static std::mutex mu;
  static size_t configured = 48 * 1024;
  {
    std::lock_guard<std::mutex> lk(mu);
    if (smem > configured) {
      if (cudaFuncSetAttribute(decode_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SMARTMEM_ERR_CUDA;
      configured = smem;
    }
  }
  profile_tick("decode_attention", st);
  // Ordinary stream ordering for this launch: started early, its thousands of small CTAs would sit on every
  // SM waiting for the GEMM before it and slow that GEMM down (measured: the step is 40 us slower).
  decode_attn_kernel<<<dim3((unsigned)(B * a.heads)), dim3(DEC_THREADS), smem, st>>>(a);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

// Explicit variant: in-place rotary embedding of rows [R, 128] that all sit at position `pos`.
__global__ void rope_rows_at_kernel(__nv_bfloat16* x, long long rows, int pos, double theta, int rot) {
  pdl_wait();
  pdl_launch_dependents();
  const int half = rot / 2;                     // pairs (i, i + rot/2) of the first rot elements of a row
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * half) return;
  const long long r = idx / half;
  const int i = (int)(idx - r * half);
  double sn, cs;
  sincos((double)pos * pow(theta, -(double)i / half), &sn, &cs);
  __nv_bfloat16* row = x + r * DH;
  const float a = __bfloat162float(row[i]), b = __bfloat162float(row[i + half]);
  row[i] = __float2bfloat16_rn(a * (float)cs - b * (float)sn);
  row[i + half] = __float2bfloat16_rn(b * (float)cs + a * (float)sn);
}

// Explicit variant: the Concat of the cache with the new rows, for a cache with room left: row r of
// src [R, 128] goes to dst + r * dst_row_stride (the slot of position `pos` of (sequence, head) r).
__global__ void append_rows_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* dst, long long rows,
                                   long long dst_row_stride) {
  pdl_wait();
  pdl_launch_dependents();
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;   // one 16-byte vector each
  if (idx >= rows * (DH / 8)) return;
  const long long r = idx / (DH / 8);
  const int v = (int)(idx - r * (DH / 8));
  *reinterpret_cast<uint4*>(dst + r * dst_row_stride + v * 8) = *reinterpret_cast<const uint4*>(src + r * DH + v * 8);
}

int launch_rope_rows_at(void* x, long long rows, int pos, float theta, int rot, cudaStream_t st) {
  const long long n = rows * (rot / 2);
  profile_tick("rope_rows", st);
  launch_pdl(rope_rows_at_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, (__nv_bfloat16*)x, rows, pos, (double)theta, rot);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

int launch_append_rows(const void* src, void* dst, long long rows, long long dst_row_stride, const char* label,
                       cudaStream_t st) {
  const long long n = rows * (DH / 8);
  profile_tick(label, st);
  launch_pdl(append_rows_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, (const __nv_bfloat16*)src,
             (__nv_bfloat16*)dst, rows, dst_row_stride);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
}

// Head split of one token per sequence: [B, 1, 3*H*D] -> [3, B, H, 1, D].
typedef std::tuple<int, int, int> DKey;
std::mutex g_mu;
std::map<DKey, smartmem_index_map_t> g_split;

int get_split(int B, int H, int D, smartmem_index_map_t* out) {   // (a copy: clearing the cache cannot invalidate it)
  DKey key(B, H, D);
  std::lock_guard<std::mutex> lk(g_mu);
  auto it = g_split.find(key);
  if (it != g_split.end()) { *out = it->second; return SMARTMEM_OK; }
  smartmem_index_map_t m;
  const int64_t b = B, h = H, d = D;
  int rc = chain_map({b, 1, 3 * h * d}, {op_reshape({b, 1, 3, h, d}), op_transpose({2, 0, 3, 1, 4})}, SMARTMEM_BF16, &m);
  if (rc != SMARTMEM_OK) return rc;
  if (g_split.size() > 64) g_split.clear();
  *out = g_split.emplace(key, m).first->second;
  return SMARTMEM_OK;
}

size_t al(size_t b) { return (b + 255) & ~(size_t)255; }

struct Layout { size_t xn, qkv, ao, split, total; };

Layout ws_layout(const smartmem_attn_params_t& p, int mode) {
  const size_t BH = al((size_t)p.B * p.hidden * 2);
  Layout L;
  memset(&L, 0, sizeof(L));
  size_t off = 0;
  auto take = [&](size_t b) { size_t o = off; off += b; return o; };
  L.xn = take(BH);
  L.qkv = take(3 * BH);        // ELIMINATE uses the first third (q only: k and v go to the caches)
  L.ao = take(BH);
  if (mode == SMARTMEM_EXPLICIT) L.split = take(3 * BH);
  L.total = off;
  return L;
}

int validate(const smartmem_attn_params_t* p, int mode) {
  if (!p) return SMARTMEM_ERR_INVALID_ARG;
  if (mode != SMARTMEM_ELIMINATE && mode != SMARTMEM_EXPLICIT) return SMARTMEM_ERR_INVALID_ARG;
  if (p->dtype != SMARTMEM_BF16) return SMARTMEM_ERR_UNSUPPORTED;
  if (p->B < 1 || p->S < 1 || p->hidden < 1 || p->heads < 1) return SMARTMEM_ERR_SHAPE;
  if (p->heads * p->head_dim != p->hidden) return SMARTMEM_ERR_SHAPE;
  if (p->head_dim != DH || p->hidden % 256) return SMARTMEM_ERR_UNSUPPORTED;
  if (p->rotary_dim != 0 && p->rotary_dim != 32 && p->rotary_dim != 64 && p->rotary_dim != 128) return SMARTMEM_ERR_UNSUPPORTED;
  return SMARTMEM_OK;
}

}  // namespace

EXPORT int smartmem_attn_decode_workspace_bytes(const smartmem_attn_params_t* p, int32_t mode, size_t* bytes) {
  int rc = validate(p, mode);
  if (rc != SMARTMEM_OK) return rc;
  if (!bytes) return SMARTMEM_ERR_INVALID_ARG;
  *bytes = ws_layout(*p, mode).total;
  return SMARTMEM_OK;
}

EXPORT int smartmem_attn_decode(const smartmem_attn_params_t* pp, int32_t pos, const void* x, void* k_cache,
                                void* v_cache, void* y, void* workspace, size_t workspace_bytes, int32_t mode,
                                void* cuda_stream) {
  int rc = validate(pp, mode);
  if (rc != SMARTMEM_OK) return rc;
  const smartmem_attn_params_t& p = *pp;
  if (pos < 0 || pos >= p.S) return SMARTMEM_ERR_SHAPE;
  if (pos + 1 > DEC_MAX_S) return SMARTMEM_ERR_UNSUPPORTED;
  if (!x || !y || !k_cache || !v_cache || !workspace || x == y || !p.rms_g || !p.w_qkv || !p.w_o)
    return SMARTMEM_ERR_INVALID_ARG;
  const void* al16[] = {x, y, k_cache, v_cache, workspace, p.rms_g, p.w_qkv, p.w_o};
  for (const void* q : al16)
    if ((uintptr_t)q & 15) return SMARTMEM_ERR_ALIGNMENT;
  const Layout L = ws_layout(p, mode);
  if (workspace_bytes < L.total) return SMARTMEM_ERR_WORKSPACE;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return SMARTMEM_ERR_CUDA;

  cudaStream_t st = (cudaStream_t)cuda_stream;
  const bool elim = mode == SMARTMEM_ELIMINATE;
  const long long B = p.B, Smax = p.S, H = p.heads, hid = p.hidden;
  char* w = (char*)workspace;
  auto at = [&](size_t off) { return (void*)(w + off); };
  __nv_bfloat16* kc = (__nv_bfloat16*)k_cache;
  __nv_bfloat16* vc = (__nv_bfloat16*)v_cache;

#define SM_TRY(expr) do { rc = (expr); if (rc != SMARTMEM_OK) return rc; } while (0)
  SM_TRY(launch_norm(SMARTMEM_BF16, true, x, at(L.xn), p.rms_g, nullptr, p.rms_eps, B, (int)hid, nullptr, st));
  DecodeAttnArgs a;
  memset(&a, 0, sizeof(a));
  a.heads = (int)H;
  a.S = pos + 1;
  a.scale_log2e = 1.4426950408889634f / sqrtf((float)DH);
  a.k = kc;
  a.v = vc;
  a.o = (__nv_bfloat16*)at(L.ao);
  a.o_sb = hid;                // [B, H, 1, D] and [B, 1, H*D] are the same bytes: the merge of one token is free
  a.o_sh = DH;
  {
    TcEpilogue ep;
    memset(&ep, 0, sizeof(ep));
    ep.out = at(L.qkv);
    ep.ldc = 3 * hid;
    if (elim) {
      ep.rope_cols = (int)(2 * hid);
      ep.rope_S = 1;
      ep.rope_pos0 = pos;
      ep.rope_log2_theta = log2f(p.rope_theta);
      ep.rope_dim = p.rotary_dim ? p.rotary_dim : DH;
      ep.seg_cols = (int)hid;
      ep.seg_out[0] = at(L.qkv);              ep.seg_ld[0] = hid;
      ep.seg_out[1] = kc + (long long)pos * hid;   ep.seg_ld[1] = Smax * hid;
      ep.seg_out[2] = vc + (long long)pos * hid;   ep.seg_ld[2] = Smax * hid;
    }
    SM_TRY(launch_gemm_tc(tc_operand_plain(at(L.xn), B, hid, hid), tc_operand_plain(p.w_qkv, 3 * hid, hid, hid), ep, 1, B,
                          3 * hid, hid, st));
  }
  if (elim) {
    a.q = (const __nv_bfloat16*)at(L.qkv);
    a.q_sb = hid; a.q_sh = DH;
    a.kv_sb = Smax * hid; a.kv_sh = DH; a.kv_ss = hid;
  } else {
    smartmem_index_map_t split;
    SM_TRY(get_split(p.B, p.heads, DH, &split));
    SM_TRY(launch_copy_map(split, 2, at(L.qkv), at(L.split), st));
    __nv_bfloat16* sp = (__nv_bfloat16*)at(L.split);
    SM_TRY(launch_rope_rows_at(sp, 2 * B * H, pos, p.rope_theta, p.rotary_dim ? p.rotary_dim : DH, st));
    SM_TRY(launch_append_rows(sp + B * hid, kc + (long long)pos * DH, B * H, Smax * DH, "append_k", st));
    SM_TRY(launch_append_rows(sp + 2 * B * hid, vc + (long long)pos * DH, B * H, Smax * DH, "append_v", st));
    a.q = sp;
    a.q_sb = hid; a.q_sh = DH;
    a.kv_sb = H * Smax * DH; a.kv_sh = Smax * DH; a.kv_ss = DH;
  }
  SM_TRY(launch_decode_attention(a, p.B, st));
  {
    TcEpilogue ep;
    memset(&ep, 0, sizeof(ep));
    ep.out = y;
    ep.ldc = hid;
    ep.residual = p.add_residual ? x : nullptr;
    SM_TRY(launch_gemm_tc(tc_operand_plain(at(L.ao), B, hid, hid), tc_operand_plain(p.w_o, hid, hid, hid), ep, 1, B, hid,
                          hid, st));
  }
#undef SM_TRY
  return SMARTMEM_OK;
}
