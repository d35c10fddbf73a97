// smartmem_swin_block: one Swin Transformer block as a fixed operator chain.
//
// ELIMINATE: LayerNorm1 reads its rows through the composed cyclic-shift + window-partition
// map, the QKV GEMM and the window attention read/write each other's buffers in place (head
// split, K transpose and head merge are strides), and the projection GEMM scatters its rows
// through the same map (window reverse + reverse shift) while adding the residual.  No layout
// operator touches memory.
// EXPLICIT: the same compute kernels with identity maps, and one copy kernel per layout
// operator (shift, partition, head split, K transpose, head merge, window reverse, unshift).
#include <map>
#include <memory>
#include <mutex>
#include <tuple>
#include <vector>

#include "attn.cuh"
#include "common.cuh"
#include "gemm_tc.cuh"
#include "chain_util.hpp"

#define EXPORT extern "C" __attribute__((visibility("default")))

using namespace smartmem;

namespace {

struct SwinMaps {
  smartmem_index_map_t e1, shift, part, split, kt, merge, rev, unshift;
  DevMap e1_rows;
};

typedef std::tuple<int, int, int, int, int, int, int, int> SwinKey;
std::mutex g_mu;
std::map<SwinKey, std::shared_ptr<const SwinMaps>> g_maps;   // entries are handed out by shared pointer: clearing the cache never invalidates a caller's copy

int get_maps(const smartmem_swin_params_t& p, std::shared_ptr<const SwinMaps>* out) {
  SwinKey key(p.dtype, p.B, p.H, p.W, p.C, p.heads, p.window, p.shift);
  std::lock_guard<std::mutex> lk(g_mu);
  auto it = g_maps.find(key);
  if (it != g_maps.end()) {
    *out = it->second;
    return SMARTMEM_OK;
  }
  SwinMaps m;
  const int64_t B = p.B, H = p.H, W = p.W, C = p.C, ws = p.window, s = p.shift, nH = p.heads, d = C / nH;
  const int64_t T = ws * ws, nW = B * (H / ws) * (W / ws);
  int rc;
  std::vector<smartmem_op_t> sh = {op_roll(1, -s), op_roll(2, -s)};
  std::vector<smartmem_op_t> e1 = sh;
  e1.push_back(op_window(SMARTMEM_OP_WINDOW_PARTITION, (int)ws));
  if ((rc = chain_map({B, H, W, C}, e1, p.dtype, &m.e1))) return rc;
  if ((rc = chain_map({B, H, W, C}, sh, p.dtype, &m.shift))) return rc;
  if ((rc = chain_map({B, H, W, C}, {op_window(SMARTMEM_OP_WINDOW_PARTITION, (int)ws)}, p.dtype, &m.part))) return rc;
  if ((rc = chain_map({nW, T, 3 * C}, {op_reshape({nW, T, 3, nH, d}), op_transpose({2, 0, 3, 1, 4})}, p.dtype, &m.split)))
    return rc;
  if ((rc = chain_map({nW, nH, T, d}, {op_transpose({0, 1, 3, 2})}, p.dtype, &m.kt))) return rc;
  if ((rc = chain_map({nW, nH, T, d}, {op_transpose({0, 2, 1, 3}), op_reshape({nW, T, C})}, p.dtype, &m.merge))) return rc;
  if ((rc = chain_map({nW, T, C}, {op_window(SMARTMEM_OP_WINDOW_REVERSE, (int)ws, B, H, W)}, p.dtype, &m.rev))) return rc;
  if ((rc = chain_map({B, H, W, C}, {op_roll(1, s), op_roll(2, s)}, p.dtype, &m.unshift))) return rc;
  // rows of the windowed [M, C] view -> offset of the token in [B,H,W,C]
  // the copy-consumer map may have merged the innermost row atom with the channel atom (no shift)
  {
    const int k = m.e1.n_atoms - 1;
    if (k >= 0 && m.e1.roll_of[k] < 0 && m.e1.src_stride[k] == 1 && m.e1.extent[k] > C && m.e1.extent[k] % C == 0 &&
        k + 1 < SMARTMEM_MAX_ATOMS) {
      m.e1.extent[k + 1] = C;
      m.e1.src_stride[k + 1] = 1;
      m.e1.roll_of[k + 1] = -1;
      m.e1.roll_weight[k + 1] = 0;
      m.e1.extent[k] /= C;
      m.e1.src_stride[k] = C;
      m.e1.n_atoms++;
    }
  }
  const int n = m.e1.n_atoms;
  if (n < 2 || m.e1.extent[n - 1] != C || m.e1.src_stride[n - 1] != 1 || m.e1.klass == 3) return SMARTMEM_ERR_UNSUPPORTED;
  if (!make_devmap(m.e1, 0, n - 1, 1, true, &m.e1_rows)) return SMARTMEM_ERR_UNSUPPORTED;
  if (g_maps.size() > 64) g_maps.clear();
  *out = g_maps.emplace(key, std::make_shared<const SwinMaps>(m)).first->second;
  return SMARTMEM_OK;
}

struct Layout {
  size_t xn, qkv, ao, y1, yn, hid, xs, xw, split, kt, oh, om, orev, ouns, total;
};

size_t al(size_t b) { return (b + 255) & ~(size_t)255; }

// Which fused kernels a block takes (they decide which intermediates exist at all).
struct Path {
  bool fuse_attn, fuse_ln1, fuse_mlp;
};
Path choose_path(const smartmem_swin_params_t& p, int mode) {
  const bool bf16 = p.dtype == SMARTMEM_BF16;
  Path t;
  t.fuse_attn = mode == SMARTMEM_ELIMINATE && swin_attn_fused_supported(p.dtype, p.C, p.heads, p.window);
  t.fuse_ln1 = bf16 && gemm_ln_supported(3 * (long long)p.C, p.C);
  t.fuse_mlp = bf16 && p.mlp_ratio > 0 && mlp_fused_supported(p.C, (long long)p.C * p.mlp_ratio);
  return t;
}

// Only the intermediates the chosen path writes are reserved.
Layout ws_layout(const smartmem_swin_params_t& p, int mode) {
  const size_t esz = p.dtype == SMARTMEM_F32 ? 4 : 2;
  const size_t MC = al((size_t)p.B * p.H * p.W * p.C * esz);
  const Path t = choose_path(p, mode);
  Layout L;
  memset(&L, 0, sizeof(L));
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += bytes; return o; };
  if (!t.fuse_attn) {
    if (!t.fuse_ln1) L.xn = take(MC);
    L.qkv = take(3 * MC);
    L.ao = take(MC);
  }
  if (p.mlp_ratio > 0) {
    L.y1 = take(MC);
    if (!t.fuse_mlp) {
      L.yn = take(MC);
      L.hid = take((size_t)p.mlp_ratio * MC);
    }
  }
  if (mode == SMARTMEM_EXPLICIT) {
    L.xs = take(MC);
    L.xw = take(MC);
    L.split = take(3 * MC);
    L.kt = take(MC);
    L.oh = take(MC);
    L.om = take(MC);
    L.orev = take(MC);
    L.ouns = take(MC);
  }
  L.total = off > 256 ? off : 256;                 // never zero: callers pass a non-null workspace
  return L;
}

int validate(const smartmem_swin_params_t* p, int mode) {
  if (!p) return SMARTMEM_ERR_INVALID_ARG;
  if (mode != SMARTMEM_ELIMINATE && mode != SMARTMEM_EXPLICIT && mode != SMARTMEM_ELIMINATE_UNFUSED) return SMARTMEM_ERR_INVALID_ARG;
  if (p->dtype != SMARTMEM_F32 && p->dtype != SMARTMEM_BF16) return SMARTMEM_ERR_UNSUPPORTED;
  if (p->B < 1 || p->H < 1 || p->W < 1 || p->C < 1 || p->heads < 1 || p->window < 1 || p->mlp_ratio < 0)
    return SMARTMEM_ERR_SHAPE;
  if (p->H % p->window || p->W % p->window || p->shift < 0 || p->shift >= p->window) return SMARTMEM_ERR_SHAPE;
  if (p->C % p->heads) return SMARTMEM_ERR_SHAPE;
  const int d = p->C / p->heads;
  if (d != 16 && d != 32) return SMARTMEM_ERR_UNSUPPORTED;
  if (p->window * p->window > 64 || p->C % 8) return SMARTMEM_ERR_UNSUPPORTED;
  return SMARTMEM_OK;
}

}  // namespace

EXPORT int smartmem_swin_block_workspace_bytes(const smartmem_swin_params_t* p, int32_t mode, size_t* bytes) {
  int rc = validate(p, mode);
  if (rc != SMARTMEM_OK) return rc;
  if (!bytes) return SMARTMEM_ERR_INVALID_ARG;
  *bytes = ws_layout(*p, mode).total;
  return SMARTMEM_OK;
}

namespace {
// Records a CUDA event before every kernel launch so that per-kernel durations can be read back.
struct KernelTimer {
  std::vector<cudaEvent_t> ev;
  std::vector<const char*> names;
  cudaStream_t st;
  void tick(const char* name) {
    cudaEvent_t e;
    cudaEventCreate(&e);
    cudaEventRecord(e, st);
    ev.push_back(e);
    names.push_back(name);
  }
};

// half: -1 the whole block, 0 the attention half only, 1 the MLP half only (x is then the attention half's result)
int run_block(const smartmem_swin_params_t* pp, const void* x, void* y, void* workspace, size_t workspace_bytes,
              int32_t mode, void* cuda_stream, KernelTimer* tm, int half = -1) {
  int rc = validate(pp, mode);
  if (rc != SMARTMEM_OK) return rc;
  if (half < -1 || half > 1 || (half == 1 && pp->mlp_ratio == 0)) return SMARTMEM_ERR_INVALID_ARG;
  const smartmem_swin_params_t& p = *pp;
  if (!x || !y || !workspace || x == y) return SMARTMEM_ERR_INVALID_ARG;
  const void* need[] = {p.ln1_g, p.ln1_b, p.w_qkv, p.b_qkv, p.rel_bias_table, p.w_proj, p.b_proj};
  for (const void* q : need)
    if (!q) return SMARTMEM_ERR_INVALID_ARG;
  const void* need2[] = {p.ln2_g, p.ln2_b, p.w_fc1, p.b_fc1, p.w_fc2, p.b_fc2};
  if (p.mlp_ratio > 0)
    for (const void* q : need2)
      if (!q) return SMARTMEM_ERR_INVALID_ARG;
  const void* al16[] = {x, y, workspace, p.ln1_g, p.ln1_b, p.w_qkv, p.b_qkv, p.w_proj, p.b_proj,
                        p.ln2_g, p.ln2_b, p.w_fc1, p.b_fc1, p.w_fc2, p.b_fc2};
  for (const void* q : al16)
    if ((uintptr_t)q & 15) return SMARTMEM_ERR_ALIGNMENT;
  const Layout L = ws_layout(p, mode);
  if (workspace_bytes < L.total) return SMARTMEM_ERR_WORKSPACE;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return SMARTMEM_ERR_CUDA;
  std::shared_ptr<const SwinMaps> mp;
  if ((rc = get_maps(p, &mp)) != SMARTMEM_OK) return rc;
  const SwinMaps& m = *mp;

  cudaStream_t st = (cudaStream_t)cuda_stream;
  const bool f32 = p.dtype == SMARTMEM_F32;
  const int esz = f32 ? 4 : 2;
  const bool elim = mode != SMARTMEM_EXPLICIT;
  const Path path = choose_path(p, mode);
  const long long C = p.C, nH = p.heads, d = C / nH, ws = p.window, T = ws * ws;
  const long long M = (long long)p.B * p.H * p.W, nW = M / T, hid = C * p.mlp_ratio;
  char* w = (char*)workspace;
  auto at = [&](size_t off) { return (void*)(w + off); };

  // out[M,N] = A[M,K] W^T + b (GELU) (+ residual), rows of out optionally scattered
  auto linear = [&](const void* A, const void* Wt, const void* b, void* out, long long N, long long K, int gelu,
                    const void* residual, const DevMap* omap) -> int {
    if (f32) {
      SimtGemmArgs g;
      memset(&g, 0, sizeof(g));
      g.A = (const float*)A; g.W = (const float*)Wt; g.bias = (const float*)b; g.residual = (const float*)residual;
      g.out = (float*)out; g.M = (int)M; g.N = (int)N; g.K = (int)K; g.lda = K; g.ldc = N; g.gelu = gelu;
      if (omap) { g.has_omap = 1; g.omap = *omap; }
      return launch_gemm_simt_f32(g, st);
    }
    TcEpilogue ep;
    memset(&ep, 0, sizeof(ep));
    ep.out = out; ep.ldc = N; ep.bias = b; ep.residual = residual; ep.gelu = gelu; ep.rowmap = omap;
    return launch_gemm_tc(tc_operand_plain(A, M, K, K), tc_operand_plain(Wt, N, K, K), ep, 1, M, N, K, st);
  };

  void* y1 = (p.mlp_ratio > 0 && half != 0) ? at(L.y1) : y;      // result of the attention half
  if (half == 1) y1 = const_cast<void*>(x);
  WinAttnArgs a;
  memset(&a, 0, sizeof(a));
  a.table = p.rel_bias_table; a.table_f32 = f32 ? 1 : 0;
  a.heads = (int)nH; a.T = (int)T; a.ws = (int)ws; a.d = (int)d; a.shift = p.shift; a.H = p.H; a.W = p.W;
  a.nWw = p.W / p.window; a.win_per_img = (p.H / p.window) * (p.W / p.window);
  a.scale = 1.0f / sqrtf((float)d);

  const bool fuse_ln1 = path.fuse_ln1;
#define SM_TRY(label, expr) do { if (tm) tm->tick(label); rc = (expr); if (rc != SMARTMEM_OK) return rc; } while (0)
  if (half == 1) {
    // MLP half only
  } else if (path.fuse_attn) {
    // narrow blocks: the whole attention half in one kernel (rows gathered and scattered through the composed map)
    SM_TRY("attn_half_fused", launch_swin_attn_fused(p, m.e1_rows, x, y1, st));
  } else if (elim) {
    if (fuse_ln1) {
      // narrow blocks: LN1, the shift o partition gather and the QKV projection in one kernel
      SM_TRY("ln1_gather_qkv_gemm", launch_gemm_ln(x, &m.e1_rows, p.ln1_g, p.ln1_b, p.ln_eps, p.w_qkv, p.b_qkv, at(L.qkv), M, 3 * C, C, st));
    } else {
      SM_TRY("ln1_gather", launch_norm(p.dtype, false, x, at(L.xn), p.ln1_g, p.ln1_b, p.ln_eps, M, (int)C, &m.e1_rows, st));
      SM_TRY("qkv_gemm", linear(at(L.xn), p.w_qkv, p.b_qkv, at(L.qkv), 3 * C, C, 0, nullptr, nullptr));
    }
    char* qkv = (char*)at(L.qkv);
    a.q = {qkv, T * 3 * C, d, 3 * C, 1};
    a.k = {qkv + C * esz, T * 3 * C, d, 3 * C, 1};
    a.v = {qkv + 2 * C * esz, T * 3 * C, d, 3 * C, 1};
    a.o = {at(L.ao), T * C, d, C, 1};
    SM_TRY("window_attention", launch_window_attention(a, p.dtype, nW, st));
    SM_TRY("proj_gemm_scatter_residual", linear(at(L.ao), p.w_proj, p.b_proj, y1, C, C, 0, x, &m.e1_rows));
  } else {
    // Same kernels as above, but every layout operator is a copy.  Where LN1 is fused into the QKV
    // kernel the copies move the raw rows and the fused kernel normalises what arrives (LayerNorm is
    // per token, so it commutes with the two token permutations); otherwise LN1 runs first.
    const void* xs = x;
    if (!fuse_ln1) {
      SM_TRY("ln1", launch_norm(p.dtype, false, x, at(L.xn), p.ln1_g, p.ln1_b, p.ln_eps, M, (int)C, nullptr, st));
      xs = at(L.xn);
    }
    if (p.shift > 0) {
      SM_TRY("copy_shift", launch_copy_map(m.shift, esz, xs, at(L.xs), st));
      xs = at(L.xs);
    }
    SM_TRY("copy_partition", launch_copy_map(m.part, esz, xs, at(L.xw), st));
    if (fuse_ln1) {
      SM_TRY("ln1_qkv_gemm", launch_gemm_ln(at(L.xw), nullptr, p.ln1_g, p.ln1_b, p.ln_eps, p.w_qkv, p.b_qkv, at(L.qkv), M, 3 * C, C, st));
    } else {
      SM_TRY("qkv_gemm", linear(at(L.xw), p.w_qkv, p.b_qkv, at(L.qkv), 3 * C, C, 0, nullptr, nullptr));
    }
    SM_TRY("copy_head_split", launch_copy_map(m.split, esz, at(L.qkv), at(L.split), st));
    char* sp = (char*)at(L.split);
    SM_TRY("copy_k_transpose", launch_copy_map(m.kt, esz, sp + (size_t)M * C * esz, at(L.kt), st));
    a.q = {sp, nH * T * d, T * d, d, 1};
    a.k = {at(L.kt), nH * T * d, T * d, 1, T};
    a.v = {sp + 2 * (size_t)M * C * esz, nH * T * d, T * d, d, 1};
    a.o = {at(L.oh), nH * T * d, T * d, d, 1};
    SM_TRY("window_attention", launch_window_attention(a, p.dtype, nW, st));
    SM_TRY("copy_head_merge", launch_copy_map(m.merge, esz, at(L.oh), at(L.om), st));
    SM_TRY("copy_window_reverse", launch_copy_map(m.rev, esz, at(L.om), at(L.orev), st));
    void* ou = at(L.orev);
    if (p.shift > 0) {
      SM_TRY("copy_unshift", launch_copy_map(m.unshift, esz, at(L.orev), at(L.ouns), st));
      ou = at(L.ouns);
    }
    SM_TRY("proj_gemm_residual", linear(ou, p.w_proj, p.b_proj, y1, C, C, 0, x, nullptr));
  }
  if (p.mlp_ratio > 0 && half != 0) {
    if (path.fuse_mlp) {
      // narrow blocks: LN2 + fc1 + GELU + fc2 + residual in one kernel; neither the normalised rows
      // nor the hidden activation leave the chip
      SM_TRY("mlp_fused_ln2_fc1_gelu_fc2_residual",
             launch_mlp_fused(y1, p.ln2_g, p.ln2_b, p.ln_eps, p.w_fc1, p.b_fc1, p.w_fc2, p.b_fc2, y, M, C, hid, st));
    } else {
      SM_TRY("ln2", launch_norm(p.dtype, false, y1, at(L.yn), p.ln2_g, p.ln2_b, p.ln_eps, M, (int)C, nullptr, st));
      SM_TRY("fc1_gemm_gelu", linear(at(L.yn), p.w_fc1, p.b_fc1, at(L.hid), hid, C, 1, nullptr, nullptr));
      SM_TRY("fc2_gemm_residual", linear(at(L.hid), p.w_fc2, p.b_fc2, y, C, hid, 0, y1, nullptr));
    }
  }
#undef SM_TRY
  if (tm) tm->tick("end");
  return SMARTMEM_OK;
}
}  // namespace

EXPORT int smartmem_swin_block(const smartmem_swin_params_t* p, const void* x, void* y, void* workspace,
                               size_t workspace_bytes, int32_t mode, void* cuda_stream) {
  return run_block(p, x, y, workspace, workspace_bytes, mode, cuda_stream, nullptr);
}

EXPORT int smartmem_swin_block_half(const smartmem_swin_params_t* p, const void* x, void* y, void* workspace,
                                    size_t workspace_bytes, int32_t mode, int32_t half, void* cuda_stream) {
  if (half != 0 && half != 1) return SMARTMEM_ERR_INVALID_ARG;
  return run_block(p, x, y, workspace, workspace_bytes, mode, cuda_stream, nullptr, half);
}

EXPORT int smartmem_swin_block_timed(const smartmem_swin_params_t* p, const void* x, void* y, void* workspace,
                                     size_t workspace_bytes, int32_t mode, void* cuda_stream, float* kernel_ms,
                                     char* kernel_names, int32_t names_stride, int32_t max_kernels,
                                     int32_t* n_kernels) {
  if (!kernel_ms || !kernel_names || !n_kernels || max_kernels < 1 || names_stride < 8) return SMARTMEM_ERR_INVALID_ARG;
  KernelTimer tm;
  tm.st = (cudaStream_t)cuda_stream;
  int rc = run_block(p, x, y, workspace, workspace_bytes, mode, cuda_stream, &tm);
  int rs = cudaStreamSynchronize(tm.st) == cudaSuccess ? SMARTMEM_OK : SMARTMEM_ERR_CUDA;
  int n = 0;
  for (size_t i = 0; i + 1 < tm.ev.size() && n < max_kernels; ++i, ++n) {
    float ms = 0.f;
    if (rs == SMARTMEM_OK) cudaEventElapsedTime(&ms, tm.ev[i], tm.ev[i + 1]);
    kernel_ms[n] = ms;
    const char* s = tm.names[i];
    int k = 0;
    while (s[k] && k < names_stride - 1) { kernel_names[n * names_stride + k] = s[k]; ++k; }
    kernel_names[n * names_stride + k] = 0;
  }
  for (cudaEvent_t e : tm.ev) cudaEventDestroy(e);
  *n_kernels = n;
  return rc != SMARTMEM_OK ? rc : rs;
}

// ---------------------------------------------------------------------------------------
// Swin block without a caller workspace.
//
// Some callers of this library cannot allocate device memory at the point where they run a
// block: code that executes inside a memory-frozen phase of a serving process (its device
// memory pool is fully committed to KV caches and activations, and a cudaMalloc there either
// fails or forces a device-wide synchronisation), plugin hosts that hand the library a stream
// and buffers but keep the allocator to themselves, and start-up paths that run before the
// host framework's allocator exists.  For them the intermediates of the block live in a
// fixed array that is part of the loaded library image on every device.
// ---------------------------------------------------------------------------------------
#define SMARTMEM_STATIC_SCRATCH_BYTES (32u << 20)
static __device__ __align__(256) unsigned char g_static_scratch[SMARTMEM_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mu;
void* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the static scratch array on the current device.  In host code the name
// g_static_scratch is only a handle for the runtime, never an address a kernel may use, so the
// address is asked for once per device (with that device current) and remembered.
int static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SMARTMEM_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_scratch_mu);
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_static_scratch) != cudaSuccess || !ptr) return SMARTMEM_ERR_CUDA;
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return SMARTMEM_OK;
}
}  // namespace

EXPORT int smartmem_swin_block_static_scratch_bytes(size_t* bytes) {
  if (!bytes) return SMARTMEM_ERR_INVALID_ARG;
  *bytes = SMARTMEM_STATIC_SCRATCH_BYTES;
  return SMARTMEM_OK;
}

EXPORT int smartmem_swin_block_noalloc(const smartmem_swin_params_t* p, const void* x, void* y, int32_t mode,
                                       void* cuda_stream) {
  int rc = validate(p, mode);
  if (rc != SMARTMEM_OK) return rc;
  if (ws_layout(*p, mode).total > SMARTMEM_STATIC_SCRATCH_BYTES) return SMARTMEM_ERR_WORKSPACE;
  void* scratch = nullptr;
  if ((rc = static_scratch(&scratch)) != SMARTMEM_OK) return rc;
  return run_block(p, x, y, scratch, SMARTMEM_STATIC_SCRATCH_BYTES, mode, cuda_stream, nullptr);
}
