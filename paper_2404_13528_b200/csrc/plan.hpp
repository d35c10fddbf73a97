// Internal planner structures shared by plan.cpp (host planner) and api.cu (launchers).
#pragma once
#include <cstdint>
#include <vector>

#include "smartmem.h"

namespace smartmem {

// One stage of the sequential ("no optimisation") index program of a layout run: the
// consumer index is pushed backwards through the stages with explicit divide / modulo.
struct SeqStage {
  int kind;                          // RESHAPE, TRANSPOSE, ROLL or SLICE
  std::vector<int64_t> in_shape, out_shape;
  std::vector<int> perm;
  int axis = 0;
  int64_t shift = 0;
  std::vector<int64_t> start;
};

struct SeqProgram {
  std::vector<SeqStage> stages;      // in chain order
  std::vector<int64_t> src_shape, src_stride;
  int64_t eval(int64_t consumer_linear) const;
};

enum StepKind { STEP_COPY = 0, STEP_LINEAR = 1, STEP_BMM_NT = 2, STEP_NORM = 3 };

// Buffer reference: >= 0 caller input index; -1 the chain output; <= -2 workspace slot (-2 - slot).
struct Step {
  int kind = STEP_COPY;
  int dtype = SMARTMEM_BF16;
  int src[2] = {0, 0};
  int dst = -1;
  int weight = -1;                   // LINEAR: caller input index of W[N,K]; NORM: of gamma[C]
  int weight2 = -1;                  // NORM: caller input index of beta[C]
  float eps = 0.f;                   // NORM
  smartmem_index_map_t map[2];
  // For GEMM-like consumers the atoms of map[] are grouped: [0, n_batch_atoms) batch,
  // then row atoms, then reduction atoms (never merged across the group boundaries).
  int n_batch_atoms[2] = {0, 0}, n_row_atoms[2] = {0, 0};
  SeqProgram seq[2];
  int64_t batch = 1, M = 0, N = 0, K = 0;
  bool is_layout_copy = false;
  int placement = 0;                 // STEP_COPY: 0 best kernel, 1 plain gather through map[0], 2 plain scatter through map[0]
};

}  // namespace smartmem

struct smartmem_plan {
  int mode = 0;
  std::vector<smartmem::Step> steps;
  std::vector<size_t> slot_bytes;    // workspace slots (EXPLICIT copies, chained consumers)
  std::vector<size_t> slot_offset;
  size_t workspace_bytes = 0;
  smartmem_tensor_desc_t out_desc;
  int n_inputs = 0;
};
