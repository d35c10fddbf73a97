// A producer with two consumers of different reduction dimensions (Section 3.2.2, "Global: layout
// selections based on reduction dimension"; the redundant-copy remark of the evaluation's discussion).
//
//   P  = X Wp^T                 X [B*S, K],  Wp [N, K]          P as a tensor [B, S, N]
//   YA = P Wa^T                 reduces over N (dimension 2)     YA [B*S, Na]
//   YB[b] = P[b]^T Wb^T         reduces over S (dimension 1)     YB [B, N, Nb],  Wb [Nb, S]
//
// The layout(s) of P come from smartmem_select_layouts with the consumers' reduction dimensions and
// the number k of dimensions that can be walked without index arithmetic:
//   k = 2  one copy [B, S, N].  On this hardware the second walkable dimension is what a TMA box
//          gives: consumer B reads the same buffer as an MN-major operand (S is its reduction
//          dimension, N contiguous), so no element is written twice.
//   k = 1  two copies: [B, S, N] for consumer A and [B, N, S] for consumer B, both written by the
//          producer's epilogue (a slower write instead of a slower read, the paper's preference).
// EXPLICIT writes the default layout and transposes it with a copy kernel for consumer B.
#include <cstring>

#include "common.cuh"
#include "gemm_tc.cuh"
#include "chain_util.hpp"
#include "plan.hpp"

using namespace smartmem;

namespace {

size_t al(size_t b) { return (b + 255) & ~(size_t)255; }

struct FanPlan {
  int n_layouts;            // copies of P the producer writes
  int layout_of_b;          // the layout consumer B reads (0: [B,S,N], 1: [B,N,S])
  int explicit_copy;        // EXPLICIT: a copy kernel writes the second layout
  size_t off_p, off_pt, total;
};

int plan_fanout(const smartmem_fanout_params_t& p, int mode, FanPlan* fp) {
  if (p.B < 1 || p.S < 1 || p.K < 1 || p.N < 1 || p.Na < 1 || p.Nb < 1) return SMARTMEM_ERR_INVALID_ARG;
  if (p.K % 8 || p.N % 8 || p.S % 8 || p.Na % 8 || p.Nb % 8) return SMARTMEM_ERR_UNSUPPORTED;   // 16-byte rows everywhere
  if (mode != SMARTMEM_ELIMINATE && mode != SMARTMEM_EXPLICIT) return SMARTMEM_ERR_INVALID_ARG;
  if (mode == SMARTMEM_ELIMINATE && p.k_contig != 1 && p.k_contig != 2) return SMARTMEM_ERR_INVALID_ARG;
  memset(fp, 0, sizeof(*fp));
  const size_t pbytes = (size_t)p.B * p.S * p.N * 2;
  if (mode == SMARTMEM_EXPLICIT) {
    fp->n_layouts = 1;
    fp->layout_of_b = 1;
    fp->explicit_copy = 1;
  } else {
    // consumer A aggregates along dimension 2 (N), consumer B along dimension 1 (S); each reads P once
    const int32_t red[2] = {2, 1};
    const int64_t weight[2] = {(int64_t)pbytes, (int64_t)pbytes};
    int32_t n_layouts = 0, perm[2 * SMARTMEM_MAX_DIMS], of[2];
    const int rc = smartmem_select_layouts(3, 2, red, weight, p.k_contig, 2, &n_layouts, perm, of);
    if (rc != SMARTMEM_OK) return rc;
    // layout 0 must be the default [B, S, N] (the tie goes to the dimension that is already innermost)
    if (perm[0] != 0 || perm[1] != 1 || perm[2] != 2 || of[0] != 0) return SMARTMEM_ERR_UNSUPPORTED;
    if (n_layouts == 2 && (perm[SMARTMEM_MAX_DIMS] != 0 || perm[SMARTMEM_MAX_DIMS + 1] != 2 || perm[SMARTMEM_MAX_DIMS + 2] != 1))
      return SMARTMEM_ERR_UNSUPPORTED;
    fp->n_layouts = n_layouts;
    fp->layout_of_b = of[1];
  }
  fp->off_p = 0;
  fp->off_pt = al(pbytes);
  fp->total = (fp->n_layouts == 2 || fp->explicit_copy) ? fp->off_pt + al(pbytes) : al(pbytes);
  return SMARTMEM_OK;
}

}  // namespace

extern "C" int smartmem_fanout_plan(const smartmem_fanout_params_t* p, int32_t mode, int32_t* n_copies_written,
                                    int32_t* layout_of_consumer_b, int64_t* producer_bytes_written,
                                    int64_t* copy_kernel_bytes, size_t* workspace_bytes) {
  if (!p) return SMARTMEM_ERR_INVALID_ARG;
  FanPlan fp;
  const int rc = plan_fanout(*p, mode, &fp);
  if (rc != SMARTMEM_OK) return rc;
  const int64_t pbytes = (int64_t)p->B * p->S * p->N * 2;
  if (n_copies_written) *n_copies_written = fp.n_layouts + fp.explicit_copy;
  if (layout_of_consumer_b) *layout_of_consumer_b = fp.layout_of_b;
  if (producer_bytes_written) *producer_bytes_written = pbytes * fp.n_layouts;
  if (copy_kernel_bytes) *copy_kernel_bytes = fp.explicit_copy ? 2 * pbytes : 0;      // read + write of the transposing copy
  if (workspace_bytes) *workspace_bytes = fp.total;
  return SMARTMEM_OK;
}

extern "C" int smartmem_fanout(const smartmem_fanout_params_t* p, const void* x, void* ya, void* yb, void* workspace,
                               size_t workspace_bytes, int32_t mode, void* cuda_stream) {
  if (!p || !x || !ya || !yb || !workspace || !p->w_p || !p->w_a || !p->w_b) return SMARTMEM_ERR_INVALID_ARG;
  FanPlan fp;
  int rc = plan_fanout(*p, mode, &fp);
  if (rc != SMARTMEM_OK) return rc;
  if (workspace_bytes < fp.total) return SMARTMEM_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const long long B = p->B, S = p->S, K = p->K, N = p->N, Na = p->Na, Nb = p->Nb;
  char* P = (char*)workspace + fp.off_p;
  char* Pt = (char*)workspace + fp.off_pt;

  // producer: P = X Wp^T, in the selected layout(s)
  {
    TcEpilogue ep;
    memset(&ep, 0, sizeof(ep));
    ep.out = P;
    ep.ldc = N;
    if (fp.n_layouts == 2) {
      ep.out2 = Pt;
      ep.out2_S = S;
    }
    rc = launch_gemm_tc(tc_operand_plain(x, B * S, K, K), tc_operand_plain(p->w_p, N, K, K), ep, 1, B * S, N, K, st);
    if (rc != SMARTMEM_OK) return rc;
  }
  if (fp.explicit_copy) {                              // the layout transformation as an operator of its own
    smartmem_index_map_t m;
    rc = chain_map({B, S, N}, {op_transpose({0, 2, 1})}, SMARTMEM_BF16, &m);
    if (rc != SMARTMEM_OK) return rc;
    rc = launch_copy_map(m, 2, P, Pt, st);
    if (rc != SMARTMEM_OK) return rc;
  }
  // consumer A: reduces over N, reads layout 0 as it lies
  {
    TcEpilogue ep;
    memset(&ep, 0, sizeof(ep));
    ep.out = ya;
    ep.ldc = Na;
    rc = launch_gemm_tc(tc_operand_plain(P, B * S, N, N), tc_operand_plain(p->w_a, Na, N, N), ep, 1, B * S, Na, N, st);
    if (rc != SMARTMEM_OK) return rc;
  }
  // consumer B: reduces over S
  {
    TcOperand A;
    memset(&A, 0, sizeof(A));
    A.n_batch_atoms = 1;
    A.batch_extent[0] = B;
    A.batch_stride[0] = S * N;
    A.n_row_atoms = 1;
    A.row_extent[0] = N;
    A.K = S;
    if (fp.layout_of_b == 0) {                         // layout 0 read with S as the reduction dimension: MN-major operand
      A.ptr = P;
      A.row_stride[0] = 1;
      A.k_stride = N;
    } else {                                           // the [B, N, S] copy, reduction dimension contiguous
      A.ptr = Pt;
      A.row_stride[0] = S;
      A.k_stride = 1;
    }
    TcEpilogue ep;
    memset(&ep, 0, sizeof(ep));
    ep.out = yb;
    ep.ldc = Nb;
    ep.out_batch_stride = N * Nb;
    rc = launch_gemm_tc(A, tc_operand_plain(p->w_b, Nb, S, S), ep, B, N, Nb, S, st);
    if (rc != SMARTMEM_OK) return rc;
  }
  return SMARTMEM_OK;
}
