// Helpers to build layout-operator chains and obtain their composed maps from the planner.
#pragma once
#include <cstring>
#include <initializer_list>
#include <vector>

#include "smartmem.h"

namespace smartmem {

inline smartmem_op_t op_reshape(std::initializer_list<int64_t> shape) {
  smartmem_op_t o;
  memset(&o, 0, sizeof(o));
  o.kind = SMARTMEM_OP_RESHAPE;
  o.ndim = (int)shape.size();
  int i = 0;
  for (int64_t v : shape) o.shape[i++] = v;
  return o;
}
inline smartmem_op_t op_transpose(std::initializer_list<int> perm) {
  smartmem_op_t o;
  memset(&o, 0, sizeof(o));
  o.kind = SMARTMEM_OP_TRANSPOSE;
  o.ndim = (int)perm.size();
  int i = 0;
  for (int v : perm) o.perm[i++] = v;
  return o;
}
inline smartmem_op_t op_roll(int axis, int64_t shift) {
  smartmem_op_t o;
  memset(&o, 0, sizeof(o));
  o.kind = SMARTMEM_OP_ROLL;
  o.axis = axis;
  o.shift = shift;
  return o;
}
inline smartmem_op_t op_window(int kind, int ws, int64_t B = 0, int64_t H = 0, int64_t W = 0) {
  smartmem_op_t o;
  memset(&o, 0, sizeof(o));
  o.kind = kind;
  o.window = ws;
  o.ndim = 3;
  o.shape[0] = B; o.shape[1] = H; o.shape[2] = W;
  return o;
}

// Composed map of a layout run on a contiguous tensor, through the planner.
inline int chain_map(std::initializer_list<int64_t> shape, std::vector<smartmem_op_t> ops, int dtype, smartmem_index_map_t* out) {
  smartmem_tensor_desc_t d;
  memset(&d, 0, sizeof(d));
  d.dtype = dtype;
  d.ndim = (int)shape.size();
  int i = 0;
  for (int64_t v : shape) d.shape[i++] = v;
  smartmem_op_t c;
  memset(&c, 0, sizeof(c));
  c.kind = SMARTMEM_OP_COPY;
  ops.push_back(c);
  smartmem_plan_t* plan = nullptr;
  int rc = smartmem_plan(ops.data(), (int)ops.size(), &d, 1, SMARTMEM_ELIMINATE, &plan);
  if (rc != SMARTMEM_OK) return rc;
  rc = smartmem_plan_get_map(plan, 0, 0, out);
  smartmem_plan_destroy(plan);
  return rc;
}


}  // namespace smartmem
