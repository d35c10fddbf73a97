// smartmem_attn_layer: one decoder attention layer (prefill) as a fixed operator chain.
//
// ELIMINATE: RMSNorm -> fused QKV GEMM whose epilogue applies the rotary embedding to the q and k
// columns -> causal attention reading q/k/v as strided boxes of the [B*S, 3*hidden] buffer (head
// split / transpose eliminated) and writing its tile at column h*D of [B*S, hidden] (head merge
// eliminated) -> output projection (+ residual).
// EXPLICIT: the same kernels with a plain QKV epilogue, a head-split copy to [3, B, H, S, D], a
// separate rotary pass over q and k, attention on the materialised tensors, a head-merge copy.
#include <map>
#include <memory>
#include <mutex>
#include <tuple>

#include "attn.cuh"
#include "chain_util.hpp"
#include "common.cuh"
#include "gemm_tc.cuh"

#define EXPORT extern "C" __attribute__((visibility("default")))

using namespace smartmem;

namespace {

struct LlamaMaps {
  smartmem_index_map_t split, merge;
};
typedef std::tuple<int, int, int, int> LKey;
std::mutex g_mu;
std::map<LKey, std::shared_ptr<const LlamaMaps>> g_maps;   // entries are handed out by shared pointer: clearing the cache never invalidates a caller's copy

int get_maps(const smartmem_attn_params_t& p, std::shared_ptr<const LlamaMaps>* out) {
  LKey key(p.B, p.S, p.heads, p.head_dim);
  std::lock_guard<std::mutex> lk(g_mu);
  auto it = g_maps.find(key);
  if (it != g_maps.end()) { *out = it->second; return SMARTMEM_OK; }
  LlamaMaps m;
  const int64_t B = p.B, S = p.S, H = p.heads, D = p.head_dim;
  int rc;
  if ((rc = chain_map({B, S, 3 * H * D}, {op_reshape({B, S, 3, H, D}), op_transpose({2, 0, 3, 1, 4})}, SMARTMEM_BF16, &m.split)))
    return rc;
  if ((rc = chain_map({B, H, S, D}, {op_transpose({0, 2, 1, 3}), op_reshape({B, S, H * D})}, SMARTMEM_BF16, &m.merge)))
    return rc;
  if (g_maps.size() > 64) g_maps.clear();
  *out = g_maps.emplace(key, std::make_shared<const LlamaMaps>(m)).first->second;
  return SMARTMEM_OK;
}

size_t al(size_t b) { return (b + 255) & ~(size_t)255; }

struct Layout { size_t xn, qkv, ao, tab, split, oh, total; };

Layout ws_layout(const smartmem_attn_params_t& p, int mode) {
  const size_t MH = al((size_t)p.B * p.S * p.hidden * 2);
  Layout L;
  memset(&L, 0, sizeof(L));
  size_t off = 0;
  auto take = [&](size_t b) { size_t o = off; off += b; return o; };
  L.xn = take(MH);
  L.qkv = take(3 * MH);
  L.ao = take(MH);
  L.tab = take(al((size_t)p.S * (p.head_dim / 2) * 8));
  if (mode == SMARTMEM_EXPLICIT) {
    L.split = take(3 * MH);
    L.oh = take(MH);
  }
  L.total = off;
  return L;
}

int validate(const smartmem_attn_params_t* p, int mode) {
  if (!p) return SMARTMEM_ERR_INVALID_ARG;
  if (mode != SMARTMEM_ELIMINATE && mode != SMARTMEM_EXPLICIT) return SMARTMEM_ERR_INVALID_ARG;
  if (p->dtype != SMARTMEM_BF16) return SMARTMEM_ERR_UNSUPPORTED;
  if (p->B < 1 || p->S < 1 || p->hidden < 1 || p->heads < 1) return SMARTMEM_ERR_SHAPE;
  if (p->heads * p->head_dim != p->hidden) return SMARTMEM_ERR_SHAPE;
  if (p->head_dim != 128 || !p->causal) return SMARTMEM_ERR_UNSUPPORTED;
  if (p->hidden % 256) return SMARTMEM_ERR_UNSUPPORTED;
  if (p->rotary_dim != 0 && p->rotary_dim != 32 && p->rotary_dim != 64 && p->rotary_dim != 128) return SMARTMEM_ERR_UNSUPPORTED;
  return SMARTMEM_OK;
}

}  // namespace

EXPORT int smartmem_attn_layer_workspace_bytes(const smartmem_attn_params_t* p, int32_t mode, size_t* bytes) {
  int rc = validate(p, mode);
  if (rc != SMARTMEM_OK) return rc;
  if (!bytes) return SMARTMEM_ERR_INVALID_ARG;
  *bytes = ws_layout(*p, mode).total;
  return SMARTMEM_OK;
}

EXPORT int smartmem_attn_layer(const smartmem_attn_params_t* pp, const void* x, void* y, void* workspace,
                               size_t workspace_bytes, int32_t mode, void* cuda_stream) {
  int rc = validate(pp, mode);
  if (rc != SMARTMEM_OK) return rc;
  const smartmem_attn_params_t& p = *pp;
  if (!x || !y || !workspace || x == y || !p.rms_g || !p.w_qkv || !p.w_o) return SMARTMEM_ERR_INVALID_ARG;
  const void* al16[] = {x, y, workspace, p.rms_g, p.w_qkv, p.w_o};
  for (const void* q : al16)
    if ((uintptr_t)q & 15) return SMARTMEM_ERR_ALIGNMENT;
  const Layout L = ws_layout(p, mode);
  if (workspace_bytes < L.total) return SMARTMEM_ERR_WORKSPACE;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return SMARTMEM_ERR_CUDA;
  std::shared_ptr<const LlamaMaps> mp;
  if ((rc = get_maps(p, &mp)) != SMARTMEM_OK) return rc;

  cudaStream_t st = (cudaStream_t)cuda_stream;
  const bool elim = mode == SMARTMEM_ELIMINATE;
  const long long S = p.S, H = p.heads, D = p.head_dim, hid = p.hidden, M = (long long)p.B * S;
  char* w = (char*)workspace;
  auto at = [&](size_t off) { return (void*)(w + off); };
  float* tab = (float*)at(L.tab);

#define SM_TRY(expr) do { rc = (expr); if (rc != SMARTMEM_OK) return rc; } while (0)
  const int rot = p.rotary_dim ? p.rotary_dim : (int)D;
  if (!elim) SM_TRY(launch_rope_table(tab, (int)S, rot, p.rope_theta, st));   // only the stand-alone RoPE pass reads it
  SM_TRY(launch_norm(SMARTMEM_BF16, true, x, at(L.xn), p.rms_g, nullptr, p.rms_eps, M, (int)hid, nullptr, st));
  {
    TcEpilogue ep;
    memset(&ep, 0, sizeof(ep));
    ep.out = at(L.qkv);
    ep.ldc = 3 * hid;
    if (elim) { ep.rope_cols = (int)(2 * hid); ep.rope_S = (int)S; ep.rope_log2_theta = log2f(p.rope_theta); ep.rope_dim = rot; }
    SM_TRY(launch_gemm_tc(tc_operand_plain(at(L.xn), M, hid, hid), tc_operand_plain(p.w_qkv, 3 * hid, hid, hid), ep, 1, M,
                          3 * hid, hid, st));
  }
  CausalAttnArgs a;
  memset(&a, 0, sizeof(a));
  a.S = (int)S; a.heads = (int)H; a.batch = p.B;
  a.scale = 1.0f / sqrtf((float)D);
  const void* proj_in;
  if (elim) {
    char* qkv = (char*)at(L.qkv);
    a.q = {qkv, S * 3 * hid, D, 3 * hid, 1};
    a.k = {qkv + hid * 2, S * 3 * hid, D, 3 * hid, 1};
    a.v = {qkv + 2 * hid * 2, S * 3 * hid, D, 3 * hid, 1};
    a.o = {at(L.ao), S * hid, D, hid, 1};
    SM_TRY(launch_causal_attention(a, st));
    proj_in = at(L.ao);
  } else {
    SM_TRY(launch_copy_map(mp->split, 2, at(L.qkv), at(L.split), st));
    char* sp = (char*)at(L.split);
    SM_TRY(launch_rope_rows(sp, 2 * M * H, (int)S, (int)D, tab, st, rot));
    const size_t one = (size_t)M * hid * 2;
    a.q = {sp, H * S * D, S * D, D, 1};
    a.k = {sp + one, H * S * D, S * D, D, 1};
    a.v = {sp + 2 * one, H * S * D, S * D, D, 1};
    a.o = {at(L.oh), H * S * D, S * D, D, 1};
    SM_TRY(launch_causal_attention(a, st));
    SM_TRY(launch_copy_map(mp->merge, 2, at(L.oh), at(L.ao), st));
    proj_in = at(L.ao);
  }
  {
    TcEpilogue ep;
    memset(&ep, 0, sizeof(ep));
    ep.out = y;
    ep.ldc = hid;
    ep.residual = p.add_residual ? x : nullptr;
    SM_TRY(launch_gemm_tc(tc_operand_plain(proj_in, M, hid, hid), tc_operand_plain(p.w_o, hid, hid, hid), ep, 1, M, hid,
                          hid, st));
  }
#undef SM_TRY
  return SMARTMEM_OK;
}
