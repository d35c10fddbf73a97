// Host-side planner: operator chain -> kernel steps with composed index maps.
//
// For every maximal run of layout operators ("Fixed output" operators, Table 3) between two
// compute operators the run is replaced by an index map evaluated inside the consumer
// (Section 3.2.1, operator elimination by index comprehension).  The map is kept in a
// canonical form built from the index dependencies the paper names -- identity (a dimension
// carried unchanged), split (a dimension factored: the "//, %" pair) and merge (factors fused:
// the "*, +" pair) -- by refining all shapes of the run to common factors ("atoms").  Because
// each atom carries its stride in the producer's buffer, every divide and modulo by a tensor
// extent cancels at plan time (the strength reduction of Section 3.2.1; the printed rule
// i % Ca % Cb = i % Cb for Cb | Ca is one instance of the cancellation), and only one modulo
// per cyclically shifted dimension survives.  The unoptimised sequential form (Fig. 4, right)
// is kept beside it for testing and for runs whose shapes do not refine.
#include "plan.hpp"

#include <algorithm>
#include <cstring>
#include <new>
#include <numeric>

namespace smartmem {

namespace {

struct Atom {
  int64_t extent, stride;
  int roll;          // -1 = plain
  int64_t weight;    // contribution of one digit step to the rolled coordinate
};
struct RollD {
  int64_t shift, mod, stride;
  std::vector<int64_t> part_extent, part_stride;   // more than one part: the rolled dim is not affine in the source
};

struct TState {
  std::vector<int64_t> shape;
  std::vector<std::vector<Atom>> dims;   // per logical dim, atoms major -> minor (extent-1 atoms dropped)
  std::vector<RollD> rolls;
  int64_t base = 0;
  bool canonical = true;
  bool fresh = true;                     // untouched contiguous buffer (a Reshape is then metadata only)
};

int64_t prod(const std::vector<int64_t>& v) {
  int64_t p = 1;
  for (int64_t x : v) p *= x;
  return p;
}

int64_t pmod(int64_t a, int64_t n) { return ((a % n) + n) % n; }

TState state_from_desc(const smartmem_tensor_desc_t& d) {
  TState s;
  bool given = false;
  for (int i = 0; i < d.ndim; ++i) given |= d.stride[i] != 0;
  int64_t run = 1;
  std::vector<int64_t> st(d.ndim);
  for (int i = d.ndim - 1; i >= 0; --i) {
    st[i] = given ? d.stride[i] : run;
    run *= d.shape[i];
  }
  bool contig = true;
  run = 1;
  for (int i = d.ndim - 1; i >= 0; --i) {
    if (d.shape[i] != 1 && st[i] != run) contig = false;
    run *= d.shape[i];
  }
  s.fresh = contig;
  for (int i = 0; i < d.ndim; ++i) {
    s.shape.push_back(d.shape[i]);
    std::vector<Atom> a;
    if (d.shape[i] > 1) a.push_back({d.shape[i], st[i], -1, 0});
    s.dims.push_back(a);
  }
  return s;
}

void do_reshape(TState& s, const std::vector<int64_t>& ns) {
  std::vector<Atom> flat;
  for (auto& d : s.dims)
    for (auto& a : d) flat.push_back(a);
  std::vector<std::vector<Atom>> nd(ns.size());
  size_t pos = 0;
  bool ok = s.canonical;
  for (size_t k = 0; k < ns.size() && ok; ++k) {
    int64_t rem = ns[k];
    while (rem > 1) {
      if (pos >= flat.size()) { ok = false; break; }
      Atom& a = flat[pos];
      if (a.extent <= rem && rem % a.extent == 0) {          // identity / merge
        nd[k].push_back(a);
        rem /= a.extent;
        ++pos;
      } else if (a.extent % rem == 0) {                        // split
        int64_t m = a.extent / rem;
        nd[k].push_back({rem, a.stride * m, a.roll, a.weight * m});
        a.extent = m;
        rem = 1;
      } else {
        ok = false;
        break;
      }
    }
  }
  s.shape = ns;
  s.dims = ok ? nd : std::vector<std::vector<Atom>>(ns.size());
  s.canonical = ok;
}

void do_transpose(TState& s, const std::vector<int>& perm) {
  std::vector<int64_t> sh(perm.size());
  std::vector<std::vector<Atom>> nd(perm.size());
  for (size_t k = 0; k < perm.size(); ++k) {
    sh[k] = s.shape[perm[k]];
    nd[k] = s.dims[perm[k]];
  }
  s.shape = sh;
  s.dims = nd;
  s.fresh = false;
}

// Are the plain atoms of one dim nested, i.e. is the dim one affine coordinate u with
// offset u * stride_last?  On success returns the per-atom weights.
bool nested_weights(const std::vector<Atom>& d, std::vector<int64_t>& w) {
  w.assign(d.size(), 1);
  for (int i = (int)d.size() - 2; i >= 0; --i) w[i] = w[i + 1] * d[i + 1].extent;
  for (size_t i = 0; i < d.size(); ++i) {
    if (d[i].roll >= 0) return false;
    if (d[i].stride != w[i] * d.back().stride) return false;
  }
  return true;
}

void do_roll(TState& s, int axis, int64_t shift) {
  s.fresh = false;
  if (!s.canonical) return;
  int64_t N = s.shape[axis];
  if (N <= 1) return;
  int64_t sp = pmod(-shift, N);                 // out[j] = in[(j + sp) mod N]
  if (sp == 0) return;
  auto& d = s.dims[axis];
  std::vector<int64_t> w;
  if (nested_weights(d, w)) {
    if ((int)s.rolls.size() >= SMARTMEM_MAX_ROLLS) { s.canonical = false; return; }
    int r = (int)s.rolls.size();
    s.rolls.push_back({sp, N, d.back().stride, {N}, {d.back().stride}});
    for (size_t i = 0; i < d.size(); ++i) { d[i].roll = r; d[i].weight = w[i]; d[i].stride = 0; }
    return;
  }
  bool all_plain = !d.empty();
  for (auto& a : d) all_plain = all_plain && a.roll < 0;
  if (all_plain && (int)d.size() <= SMARTMEM_MAX_ROLLS && (int)s.rolls.size() < SMARTMEM_MAX_ROLLS) {
    // merged from factors that do not nest in the source: the rolled coordinate is decomposed
    // again over these factors after the wrap
    int r = (int)s.rolls.size();
    RollD rd{sp, N, 0, {}, {}};
    for (auto& a : d) { rd.part_extent.push_back(a.extent); rd.part_stride.push_back(a.stride); }
    s.rolls.push_back(rd);
    for (size_t i = 0; i < d.size(); ++i) { d[i].roll = r; d[i].weight = w[i]; d[i].stride = 0; }
    return;
  }
  // the dim is already exactly one rolled coordinate: shifts add
  int r = d.empty() ? -1 : d[0].roll;
  bool same = r >= 0 && s.rolls[r].mod == N;
  int64_t ww = 1;
  for (int i = (int)d.size() - 1; i >= 0 && same; --i) {
    same = d[i].roll == r && d[i].weight == ww;
    ww *= d[i].extent;
  }
  if (same && ww == N) {
    s.rolls[r].shift = pmod(s.rolls[r].shift + sp, N);
    return;
  }
  s.canonical = false;
}

void do_slice(TState& s, const std::vector<int64_t>& start, const std::vector<int64_t>& ext) {
  for (size_t k = 0; k < s.shape.size(); ++k) {
    if (start[k] == 0 && ext[k] == s.shape[k]) continue;
    s.fresh = false;
    if (s.canonical) {
      auto& d = s.dims[k];
      std::vector<int64_t> w;
      if (d.size() > 1 && nested_weights(d, w)) {      // merge nested plain atoms back into one
        Atom m{s.shape[k], d.back().stride, -1, 0};
        d.assign(1, m);
      }
      if (d.size() == 1 && d[0].roll < 0) {
        s.base += start[k] * d[0].stride;
        d[0].extent = ext[k];
      } else if (d.size() == 1) {
        RollD& r = s.rolls[d[0].roll];
        r.shift = pmod(r.shift + start[k] * d[0].weight, r.mod);
        d[0].extent = ext[k];
      } else {
        s.canonical = false;
      }
      if (ext[k] == 1) d.clear();
    }
    s.shape[k] = ext[k];
  }
}

// Appends the primitive stages of one layout operator to `seq` and applies them to `s`.
int apply_layout_op(const smartmem_op_t& op, TState& s, SeqProgram& seq) {
  auto push = [&](SeqStage st) {
    st.in_shape = s.shape;
    switch (st.kind) {
      case SMARTMEM_OP_RESHAPE: do_reshape(s, st.out_shape); break;
      case SMARTMEM_OP_TRANSPOSE: do_transpose(s, st.perm); break;
      case SMARTMEM_OP_ROLL: do_roll(s, st.axis, st.shift); break;
      case SMARTMEM_OP_SLICE: do_slice(s, st.start, st.out_shape); break;
    }
    st.out_shape = s.shape;
    seq.stages.push_back(st);
  };
  const int nd = (int)s.shape.size();
  switch (op.kind) {
    case SMARTMEM_OP_RESHAPE: {
      if (op.ndim < 1 || op.ndim > SMARTMEM_MAX_DIMS) return SMARTMEM_ERR_INVALID_ARG;
      SeqStage st;
      st.kind = SMARTMEM_OP_RESHAPE;
      st.out_shape.assign(op.shape, op.shape + op.ndim);
      for (int64_t e : st.out_shape)
        if (e < 1) return SMARTMEM_ERR_SHAPE;
      if (prod(st.out_shape) != prod(s.shape)) return SMARTMEM_ERR_SHAPE;
      push(st);
      return SMARTMEM_OK;
    }
    case SMARTMEM_OP_TRANSPOSE: {
      if (op.ndim != nd) return SMARTMEM_ERR_SHAPE;
      SeqStage st;
      st.kind = SMARTMEM_OP_TRANSPOSE;
      st.perm.assign(op.perm, op.perm + nd);
      std::vector<int> chk(st.perm);
      std::sort(chk.begin(), chk.end());
      for (int i = 0; i < nd; ++i)
        if (chk[i] != i) return SMARTMEM_ERR_SHAPE;
      push(st);
      return SMARTMEM_OK;
    }
    case SMARTMEM_OP_ROLL: {
      if (op.axis < 0 || op.axis >= nd) return SMARTMEM_ERR_SHAPE;
      SeqStage st;
      st.kind = SMARTMEM_OP_ROLL;
      st.axis = op.axis;
      st.shift = op.shift;
      push(st);
      return SMARTMEM_OK;
    }
    case SMARTMEM_OP_SLICE: {
      if (op.ndim != nd) return SMARTMEM_ERR_SHAPE;
      SeqStage st;
      st.kind = SMARTMEM_OP_SLICE;
      st.start.assign(op.start, op.start + nd);
      st.out_shape.assign(op.shape, op.shape + nd);
      for (int i = 0; i < nd; ++i)
        if (st.start[i] < 0 || st.out_shape[i] < 1 || st.start[i] + st.out_shape[i] > s.shape[i])
          return SMARTMEM_ERR_SHAPE;
      push(st);
      return SMARTMEM_OK;
    }
    case SMARTMEM_OP_WINDOW_PARTITION: {
      if (nd != 4 || op.window < 1) return SMARTMEM_ERR_SHAPE;
      int64_t B = s.shape[0], H = s.shape[1], W = s.shape[2], C = s.shape[3], ws = op.window;
      if (H % ws || W % ws) return SMARTMEM_ERR_SHAPE;
      SeqStage a, b, c;
      a.kind = SMARTMEM_OP_RESHAPE;
      a.out_shape = {B, H / ws, ws, W / ws, ws, C};
      b.kind = SMARTMEM_OP_TRANSPOSE;
      b.perm = {0, 1, 3, 2, 4, 5};
      c.kind = SMARTMEM_OP_RESHAPE;
      c.out_shape = {B * (H / ws) * (W / ws), ws * ws, C};
      push(a); push(b); push(c);
      return SMARTMEM_OK;
    }
    case SMARTMEM_OP_WINDOW_REVERSE: {
      if (nd != 3 || op.window < 1 || op.ndim < 3) return SMARTMEM_ERR_SHAPE;
      int64_t B = op.shape[0], H = op.shape[1], W = op.shape[2], C = s.shape[2], ws = op.window;
      if (B < 1 || H < 1 || W < 1 || H % ws || W % ws) return SMARTMEM_ERR_SHAPE;
      if (s.shape[0] != B * (H / ws) * (W / ws) || s.shape[1] != ws * ws) return SMARTMEM_ERR_SHAPE;
      SeqStage a, b, c;
      a.kind = SMARTMEM_OP_RESHAPE;
      a.out_shape = {B, H / ws, W / ws, ws, ws, C};
      b.kind = SMARTMEM_OP_TRANSPOSE;
      b.perm = {0, 1, 3, 2, 4, 5};
      c.kind = SMARTMEM_OP_RESHAPE;
      c.out_shape = {B, H, W, C};
      push(a); push(b); push(c);
      return SMARTMEM_OK;
    }
    case SMARTMEM_OP_DEPTH_TO_SPACE: {
      if (nd != 4 || op.window < 1) return SMARTMEM_ERR_SHAPE;
      int64_t N = s.shape[0], Cb = s.shape[1], H = s.shape[2], W = s.shape[3], b = op.window;
      if (Cb % (b * b)) return SMARTMEM_ERR_SHAPE;
      SeqStage x, y, z;
      x.kind = SMARTMEM_OP_RESHAPE;
      x.out_shape = {N, b, b, Cb / (b * b), H, W};
      y.kind = SMARTMEM_OP_TRANSPOSE;
      y.perm = {0, 3, 4, 1, 5, 2};
      z.kind = SMARTMEM_OP_RESHAPE;
      z.out_shape = {N, Cb / (b * b), H * b, W * b};
      push(x); push(y); push(z);
      return SMARTMEM_OK;
    }
    case SMARTMEM_OP_SPACE_TO_DEPTH: {
      if (nd != 4 || op.window < 1) return SMARTMEM_ERR_SHAPE;
      int64_t N = s.shape[0], C = s.shape[1], H = s.shape[2], W = s.shape[3], b = op.window;
      if (H % b || W % b) return SMARTMEM_ERR_SHAPE;
      SeqStage x, y, z;
      x.kind = SMARTMEM_OP_RESHAPE;
      x.out_shape = {N, C, H / b, b, W / b, b};
      y.kind = SMARTMEM_OP_TRANSPOSE;
      y.perm = {0, 3, 5, 1, 2, 4};
      z.kind = SMARTMEM_OP_RESHAPE;
      z.out_shape = {N, C * b * b, H / b, W / b};
      push(x); push(y); push(z);
      return SMARTMEM_OK;
    }
  }
  return SMARTMEM_ERR_INVALID_ARG;
}

bool moves_data(int kind) { return kind != SMARTMEM_OP_RESHAPE; }

// Flattens the state into the public map.  `group_end[g]` = index one past the last logical
// dim of group g; atoms are merged inside a group only.
int finalize_map(const TState& s, const std::vector<int>& group_end, int elem_size,
                 smartmem_index_map_t* m, int* atoms_per_group) {
  std::memset(m, 0, sizeof(*m));
  m->n_elements = prod(s.shape);
  m->base = s.base;
  m->vec_elems = 1;
  for (size_t g = 0; g < group_end.size(); ++g) atoms_per_group[g] = 0;
  if (!s.canonical) {
    m->klass = 3;
    return SMARTMEM_OK;
  }
  std::vector<Atom> out;
  std::vector<int> gid;
  int dim0 = 0;
  for (size_t g = 0; g < group_end.size(); ++g) {
    size_t first = out.size();
    for (int k = dim0; k < group_end[g]; ++k)
      for (Atom a : s.dims[k]) {
        if (a.extent == 1) continue;
        if (a.roll >= 0 && s.rolls[a.roll].shift == 0 && s.rolls[a.roll].part_extent.size() == 1) {   // shifts cancelled: a plain affine atom again
          a.stride = a.weight * s.rolls[a.roll].stride;
          a.roll = -1;
          a.weight = 0;
        }
        if (out.size() > first) {
          Atom& p = out.back();
          bool mp = p.roll < 0 && a.roll < 0 && p.stride == a.extent * a.stride;
          bool mr = p.roll >= 0 && p.roll == a.roll && p.weight == a.extent * a.weight;
          if (mp || mr) {
            p.extent *= a.extent;
            p.stride = a.stride;
            p.weight = a.weight;
            continue;
          }
        }
        out.push_back(a);
        gid.push_back((int)g);
      }
    atoms_per_group[g] = (int)(out.size() - first);
    dim0 = group_end[g];
  }
  if (out.size() > SMARTMEM_MAX_ATOMS) return SMARTMEM_ERR_UNSUPPORTED;
  // drop rolls that lost all their atoms (e.g. sliced to extent 1): fold into base
  std::vector<int> used(s.rolls.size(), 0), remap(s.rolls.size(), -1);
  for (auto& a : out)
    if (a.roll >= 0) used[a.roll] = 1;
  for (size_t r = 0; r < s.rolls.size(); ++r) {
    if (used[r]) {
      remap[r] = m->n_rolls;
      m->roll_shift[m->n_rolls] = s.rolls[r].shift;
      m->roll_mod[m->n_rolls] = s.rolls[r].mod;
      m->roll_stride[m->n_rolls] = s.rolls[r].stride;
      m->roll_n_parts[m->n_rolls] = (int)s.rolls[r].part_extent.size();
      for (size_t k = 0; k < s.rolls[r].part_extent.size(); ++k) {
        m->roll_part_extent[m->n_rolls][k] = s.rolls[r].part_extent[k];
        m->roll_part_stride[m->n_rolls][k] = s.rolls[r].part_stride[k];
      }
      ++m->n_rolls;
    } else {
      int64_t v = pmod(s.rolls[r].shift, s.rolls[r].mod);
      for (int k = (int)s.rolls[r].part_extent.size() - 1; k >= 0; --k) {
        m->base += (v % s.rolls[r].part_extent[k]) * s.rolls[r].part_stride[k];
        v /= s.rolls[r].part_extent[k];
      }
    }
  }
  m->n_atoms = (int)out.size();
  for (size_t i = 0; i < out.size(); ++i) {
    m->extent[i] = out[i].extent;
    m->src_stride[i] = out[i].roll < 0 ? out[i].stride : 0;
    m->roll_of[i] = out[i].roll < 0 ? -1 : remap[out[i].roll];
    m->roll_weight[i] = out[i].roll < 0 ? 0 : out[i].weight;
  }
  // widest vector: innermost atom plain with stride 1; everything else a multiple of it
  int maxv = 16 / elem_size;
  int v = 1;
  if (m->n_atoms > 0 && m->roll_of[m->n_atoms - 1] < 0 && m->src_stride[m->n_atoms - 1] == 1) {
    v = maxv;
    auto shrink = [&](int64_t q) {
      while (v > 1 && (q % v) != 0) v >>= 1;
    };
    shrink(m->extent[m->n_atoms - 1]);
    shrink(m->base);
    for (int i = 0; i + 1 < m->n_atoms; ++i)
      if (m->roll_of[i] < 0) shrink(m->src_stride[i]);
    for (int r = 0; r < m->n_rolls; ++r)
      for (int k = 0; k < m->roll_n_parts[r]; ++k) shrink(m->roll_part_stride[r][k]);
  }
  m->vec_elems = v;
  if (m->n_rolls > 0) {
    m->klass = 2;
  } else {
    bool ident = m->base == 0;
    int64_t run = 1;
    for (int i = m->n_atoms - 1; i >= 0 && ident; --i) {
      ident = m->src_stride[i] == run;
      run *= m->extent[i];
    }
    m->klass = ident ? 0 : 1;
  }
  return SMARTMEM_OK;
}

}  // namespace

int64_t SeqProgram::eval(int64_t idx) const {
  // push the consumer index backwards through the stages, one divide/modulo chain per stage
  std::vector<int64_t> c, in;
  for (int si = (int)stages.size() - 1; si >= 0; --si) {
    const SeqStage& st = stages[si];
    const int no = (int)st.out_shape.size(), ni = (int)st.in_shape.size();
    c.assign(no, 0);
    for (int k = no - 1; k >= 0; --k) {
      c[k] = idx % st.out_shape[k];
      idx /= st.out_shape[k];
    }
    in.assign(ni, 0);
    switch (st.kind) {
      case SMARTMEM_OP_RESHAPE: {
        int64_t lin = 0;
        for (int k = 0; k < no; ++k) lin = lin * st.out_shape[k] + c[k];
        idx = lin;
        continue;
      }
      case SMARTMEM_OP_TRANSPOSE:
        for (int k = 0; k < no; ++k) in[st.perm[k]] = c[k];
        break;
      case SMARTMEM_OP_ROLL:
        in = c;
        in[st.axis] = pmod(c[st.axis] - st.shift, st.in_shape[st.axis]);
        break;
      case SMARTMEM_OP_SLICE:
        for (int k = 0; k < no; ++k) in[k] = c[k] + st.start[k];
        break;
    }
    int64_t lin = 0;
    for (int k = 0; k < ni; ++k) lin = lin * st.in_shape[k] + in[k];
    idx = lin;
  }
  int64_t off = 0;
  for (int k = (int)src_shape.size() - 1; k >= 0; --k) {
    off += (idx % src_shape[k]) * src_stride[k];
    idx /= src_shape[k];
  }
  return off;
}

}  // namespace smartmem

using namespace smartmem;

namespace {

SeqProgram seq_from_desc(const smartmem_tensor_desc_t& d) {
  SeqProgram q;
  bool given = false;
  for (int i = 0; i < d.ndim; ++i) given |= d.stride[i] != 0;
  q.src_shape.assign(d.shape, d.shape + d.ndim);
  q.src_stride.resize(d.ndim);
  int64_t run = 1;
  for (int i = d.ndim - 1; i >= 0; --i) {
    q.src_stride[i] = given ? d.stride[i] : run;
    run *= d.shape[i];
  }
  return q;
}

smartmem_tensor_desc_t contiguous_desc(const std::vector<int64_t>& shape, int dtype) {
  smartmem_tensor_desc_t d;
  std::memset(&d, 0, sizeof(d));
  d.dtype = dtype;
  d.ndim = (int)shape.size();
  for (int i = 0; i < d.ndim; ++i) d.shape[i] = shape[i];
  return d;
}

struct RunResult {
  TState state;
  SeqProgram seq;
  int src;   // buffer reference of the tensor the final map reads from
};

int new_slot(smartmem_plan_t* p, int64_t elems, int esz) {
  size_t b = ((size_t)elems * esz + 255) & ~(size_t)255;
  p->slot_bytes.push_back(b);
  return -2 - (int)(p->slot_bytes.size() - 1);
}

// Runs layout operators ops[i0, i1) on the tensor `desc` living in buffer `src`.
// ELIMINATE: pure composition.  EXPLICIT: one copy step per data-moving operator.
int process_run(smartmem_plan_t* p, const smartmem_op_t* ops, int i0, int i1, const smartmem_tensor_desc_t& desc,
                int src, int mode, int esz, RunResult* out) {
  out->state = state_from_desc(desc);
  out->seq = seq_from_desc(desc);
  out->src = src;
  for (int i = i0; i < i1; ++i) {
    int rc = apply_layout_op(ops[i], out->state, out->seq);
    if (rc != SMARTMEM_OK) return rc;
    if ((int)out->state.shape.size() > SMARTMEM_MAX_DIMS) return SMARTMEM_ERR_UNSUPPORTED;
    if (mode == SMARTMEM_EXPLICIT && (moves_data(ops[i].kind) || !out->state.fresh)) {
      // materialise what has been composed so far (one operator, plus reshapes of a strided input)
      Step st;
      st.kind = STEP_COPY;
      st.dtype = desc.dtype;
      st.is_layout_copy = true;
      st.src[0] = out->src;
      std::vector<int> ge{(int)out->state.shape.size()};
      int apg[1];
      rc = finalize_map(out->state, ge, esz, &st.map[0], apg);
      if (rc != SMARTMEM_OK) return rc;
      st.seq[0] = out->seq;
      st.dst = new_slot(p, st.map[0].n_elements, esz);
      p->steps.push_back(st);
      smartmem_tensor_desc_t nd = contiguous_desc(out->state.shape, desc.dtype);
      out->state = state_from_desc(nd);
      out->seq = seq_from_desc(nd);
      out->src = st.dst;
    }
  }
  return SMARTMEM_OK;
}

// The map of a LayerNorm over a dimension that is strided in the producer while the tokens are contiguous
// ([images] x [tokens] x [C]: a channels-first producer).  Must agree with the kernel-side check in norm.cu.
bool layernorm_strided_form(const smartmem_index_map_t& m, int elem_size, int64_t C) {
  const int n = m.n_atoms;
  if (m.klass != 1 || elem_size != 2 || n < 2 || n > 3 || C % 2 || C > 512) return false;
  if (m.extent[n - 1] != C || m.src_stride[n - 1] == 1 || m.src_stride[n - 2] != 1 || m.extent[n - 2] % 64) return false;
  if (m.base % 2 || m.src_stride[n - 1] % 2 || (n == 3 && m.src_stride[0] % 2)) return false;
  return m.n_elements / C / 64 < (1ll << 31);
}

bool is_layout_kind(int k) { return k >= SMARTMEM_OP_RESHAPE && k <= SMARTMEM_OP_SPACE_TO_DEPTH; }

}  // namespace

extern "C" {

int smartmem_op_quadrant(int32_t kind, int32_t* q) {
  if (!q) return SMARTMEM_ERR_INVALID_ARG;
  switch (kind) {
    case SMARTMEM_OP_LINEAR: case SMARTMEM_OP_BMM_NT: case SMARTMEM_OP_LAYERNORM: *q = 0; return SMARTMEM_OK;   // MatMul, LayerNorm
    case SMARTMEM_OP_COPY: *q = 1; return SMARTMEM_OK;                                       // Unary (identity)
    case SMARTMEM_OP_RESHAPE: case SMARTMEM_OP_TRANSPOSE: case SMARTMEM_OP_WINDOW_PARTITION:
    case SMARTMEM_OP_WINDOW_REVERSE: case SMARTMEM_OP_DEPTH_TO_SPACE: case SMARTMEM_OP_SPACE_TO_DEPTH:
      *q = 2; return SMARTMEM_OK;                                                             // Reshape / Transpose / DtoS / StoD
    case SMARTMEM_OP_ROLL: case SMARTMEM_OP_SLICE: *q = 3; return SMARTMEM_OK;               // Gather / Slice
  }
  return SMARTMEM_ERR_INVALID_ARG;
}

int smartmem_pair_decision(int32_t a, int32_t b, int32_t* action, int32_t* result, int32_t* search) {
  if (a < 0 || a > 3 || b < 0 || b > 3 || !action || !result || !search) return SMARTMEM_ERR_INVALID_ARG;
  const bool fa = a >= 2, fb = b >= 2;     // Fixed-output operators
  if (fa && fb) {                          // eliminate both
    *action = 4; *result = -1; *search = 0;
  } else if (fa) {                         // eliminate 1st; the preserved operator decides
    *action = 2; *result = b; *search = (b == 0) ? 4 : 0;
  } else if (fb) {                         // eliminate 2nd
    *action = 3; *result = a; *search = (a == 0) ? 3 : 0;
  } else if (a == 0 && b == 0) {           // two layout-sensitive compute operators
    *action = 0; *result = 0; *search = 1;
  } else {                                 // try fuse; the more complex operator decides
    *action = 1; *result = (a == 0 || b == 0) ? 0 : 1; *search = (*result == 0) ? 2 : 0;
  }
  return SMARTMEM_OK;
}

int smartmem_select_layouts(int32_t ndim, int32_t n_consumers, const int32_t* reduction_dim, const int64_t* weight,
                            int32_t k, int32_t max_layouts, int32_t* n_layouts, int32_t* perm, int32_t* layout_of_consumer) {
  if (!reduction_dim || !n_layouts || !perm || !layout_of_consumer) return SMARTMEM_ERR_INVALID_ARG;
  if (ndim < 1 || ndim > SMARTMEM_MAX_DIMS || n_consumers < 1 || k < 1 || k > ndim || max_layouts < 1)
    return SMARTMEM_ERR_INVALID_ARG;
  int64_t demand[SMARTMEM_MAX_DIMS] = {0};
  for (int c = 0; c < n_consumers; ++c) {
    if (reduction_dim[c] >= ndim || reduction_dim[c] < -1) return SMARTMEM_ERR_INVALID_ARG;
    const int64_t w = weight ? weight[c] : 1;
    if (w <= 0) return SMARTMEM_ERR_INVALID_ARG;
    if (reduction_dim[c] >= 0) demand[reduction_dim[c]] += w;
  }
  // demanded dimensions, most demanded first; ties: the one nearer the contiguous end of the natural order
  std::vector<int> order;
  for (int d = 0; d < ndim; ++d)
    if (demand[d] > 0) order.push_back(d);
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return demand[a] != demand[b] ? demand[a] > demand[b] : a > b; });
  const int need = order.empty() ? 1 : (int)((order.size() + k - 1) / k);
  if (need > max_layouts) return SMARTMEM_ERR_UNSUPPORTED;
  int layout_of_dim[SMARTMEM_MAX_DIMS];
  for (int d = 0; d < ndim; ++d) layout_of_dim[d] = -1;
  for (int l = 0; l < need; ++l) {
    std::vector<int> inner;                                   // this layout's served dimensions, most demanded first
    for (int i = l * k; i < (l + 1) * k && i < (int)order.size(); ++i) {
      inner.push_back(order[i]);
      layout_of_dim[order[i]] = l;
    }
    int p = 0;
    for (int d = 0; d < ndim; ++d)
      if (std::find(inner.begin(), inner.end(), d) == inner.end()) perm[l * SMARTMEM_MAX_DIMS + p++] = d;
    for (int i = (int)inner.size() - 1; i >= 0; --i) perm[l * SMARTMEM_MAX_DIMS + p++] = inner[i];   // most demanded last = contiguous
    for (; p < SMARTMEM_MAX_DIMS; ++p) perm[l * SMARTMEM_MAX_DIMS + p] = -1;
  }
  for (int c = 0; c < n_consumers; ++c) layout_of_consumer[c] = reduction_dim[c] < 0 ? 0 : layout_of_dim[reduction_dim[c]];
  *n_layouts = need;
  return SMARTMEM_OK;
}

// Copy-only chains with the eliminated map placed explicitly on one side of the copy
// (Section 3.2.2: a sub-optimal write is preferred to a sub-optimal read).  GATHER composes the chain
// as usual and pins the plain map-driven kernel: out[i] = in[map(i)].  SCATTER inverts the chain
// (operators in reverse order, each replaced by its inverse), composes THAT from the output tensor's
// point of view, and obtains for every input element the output offset it goes to: out[imap(i)] = in[i].
static int plan_placement(const smartmem_op_t* ops, int32_t n_ops, const smartmem_tensor_desc_t* inputs, int32_t n_inputs,
                          int32_t mode, smartmem_plan_t** out_plan) {
  if (n_ops < 2 || ops[n_ops - 1].kind != SMARTMEM_OP_COPY || n_inputs != 1) return SMARTMEM_ERR_UNSUPPORTED;
  for (int i = 0; i + 1 < n_ops; ++i)
    if (!is_layout_kind(ops[i].kind)) return SMARTMEM_ERR_UNSUPPORTED;
  smartmem_plan_t* fwd = nullptr;
  int rc = smartmem_plan(ops, n_ops, inputs, n_inputs, SMARTMEM_ELIMINATE, &fwd);
  if (rc != SMARTMEM_OK) return rc;
  // both placements run the strength-reduced map; chains that only the sequential program can evaluate are not covered
  if (fwd->steps.size() != 1 || fwd->steps[0].kind != STEP_COPY || fwd->steps[0].map[0].klass == 3) { delete fwd; return SMARTMEM_ERR_UNSUPPORTED; }
  if (mode == SMARTMEM_ELIMINATE_GATHER) {
    fwd->mode = mode;
    fwd->steps[0].placement = 1;
    *out_plan = fwd;
    return SMARTMEM_OK;
  }
  if (!state_from_desc(inputs[0]).fresh) { delete fwd; return SMARTMEM_ERR_UNSUPPORTED; }   // the scatter walks the input linearly
  // invert the stages the forward composition went through (window operators are already expanded)
  std::vector<smartmem_op_t> inv;
  const auto& stages = fwd->steps[0].seq[0].stages;
  for (int k = (int)stages.size() - 1; k >= 0 && rc == SMARTMEM_OK; --k) {
    const SeqStage& sg = stages[k];
    smartmem_op_t o;
    memset(&o, 0, sizeof(o));
    o.kind = sg.kind;
    if (sg.kind == SMARTMEM_OP_RESHAPE) {
      o.ndim = (int)sg.in_shape.size();
      for (int d = 0; d < o.ndim; ++d) o.shape[d] = sg.in_shape[d];
    } else if (sg.kind == SMARTMEM_OP_TRANSPOSE) {
      o.ndim = (int)sg.perm.size();
      for (int d = 0; d < o.ndim; ++d) o.perm[sg.perm[d]] = d;
    } else if (sg.kind == SMARTMEM_OP_ROLL) {
      o.axis = sg.axis;
      o.shift = -sg.shift;
    } else {
      rc = SMARTMEM_ERR_UNSUPPORTED;                 // a Slice drops elements: no inverse
    }
    inv.push_back(o);
  }
  smartmem_op_t cp;
  memset(&cp, 0, sizeof(cp));
  cp.kind = SMARTMEM_OP_COPY;
  inv.push_back(cp);
  smartmem_plan_t* bwd = nullptr;
  const smartmem_tensor_desc_t out_desc = fwd->out_desc;
  delete fwd;
  if (rc != SMARTMEM_OK) return rc;
  rc = smartmem_plan(inv.data(), (int)inv.size(), &out_desc, 1, SMARTMEM_ELIMINATE, &bwd);
  if (rc != SMARTMEM_OK) return rc;
  if (bwd->steps.size() != 1 || bwd->steps[0].kind != STEP_COPY || bwd->steps[0].map[0].klass == 3) { delete bwd; return SMARTMEM_ERR_UNSUPPORTED; }
  bwd->mode = mode;
  bwd->steps[0].placement = 2;       // map[0]: input linear index -> output offset
  bwd->out_desc = out_desc;
  *out_plan = bwd;
  return SMARTMEM_OK;
}

int smartmem_plan(const smartmem_op_t* ops, int32_t n_ops, const smartmem_tensor_desc_t* inputs, int32_t n_inputs,
                  int32_t mode, smartmem_plan_t** out_plan) {
  if (!ops || !inputs || !out_plan || n_ops < 1 || n_inputs < 1) return SMARTMEM_ERR_INVALID_ARG;
  if (mode != SMARTMEM_ELIMINATE && mode != SMARTMEM_EXPLICIT && mode != SMARTMEM_ELIMINATE_NAIVE &&
      mode != SMARTMEM_ELIMINATE_GATHER && mode != SMARTMEM_ELIMINATE_SCATTER)
    return SMARTMEM_ERR_INVALID_ARG;
  if (mode == SMARTMEM_ELIMINATE_GATHER || mode == SMARTMEM_ELIMINATE_SCATTER)
    return plan_placement(ops, n_ops, inputs, n_inputs, mode, out_plan);
  for (int i = 0; i < n_inputs; ++i) {
    if (inputs[i].ndim < 1 || inputs[i].ndim > SMARTMEM_MAX_DIMS) return SMARTMEM_ERR_INVALID_ARG;
    if (inputs[i].dtype != SMARTMEM_F32 && inputs[i].dtype != SMARTMEM_BF16) return SMARTMEM_ERR_INVALID_ARG;
    for (int k = 0; k < inputs[i].ndim; ++k)
      if (inputs[i].shape[k] < 1) return SMARTMEM_ERR_SHAPE;
  }
  if (is_layout_kind(ops[n_ops - 1].kind)) return SMARTMEM_ERR_INVALID_ARG;   // must end in a consumer
  smartmem_plan_t* p = new (std::nothrow) smartmem_plan_t();
  if (!p) return SMARTMEM_ERR_INVALID_ARG;
  p->mode = mode;
  p->n_inputs = n_inputs;
  const int dtype = inputs[0].dtype;
  const int esz = dtype == SMARTMEM_F32 ? 4 : 2;
  smartmem_tensor_desc_t cur = inputs[0];
  int cur_src = 0;
  int rc = SMARTMEM_OK;
  int i = 0;
  while (i < n_ops && rc == SMARTMEM_OK) {
    int j = i;
    while (j < n_ops && is_layout_kind(ops[j].kind)) ++j;
    const smartmem_op_t& c = ops[j];
    const bool last = (j == n_ops - 1);
    RunResult A;
    rc = process_run(p, ops, i, j, cur, cur_src, mode, esz, &A);
    if (rc != SMARTMEM_OK) break;
    Step st;
    st.dtype = dtype;
    st.src[0] = A.src;
    st.seq[0] = A.seq;
    const int nd = (int)A.state.shape.size();
    std::vector<int64_t> oshape;
    int apg[3];
    if (c.kind == SMARTMEM_OP_COPY) {
      st.kind = STEP_COPY;
      rc = finalize_map(A.state, {nd}, esz, &st.map[0], apg);
      oshape = A.state.shape;
    } else if (c.kind == SMARTMEM_OP_LINEAR) {
      st.kind = STEP_LINEAR;
      int wi = c.side_input[0];
      if (wi < 1 || wi >= n_inputs) { rc = SMARTMEM_ERR_INVALID_ARG; break; }
      const smartmem_tensor_desc_t& w = inputs[wi];
      if (nd < 2) { rc = SMARTMEM_ERR_SHAPE; break; }
      if (w.ndim != 2 || w.shape[1] != A.state.shape[nd - 1] || w.dtype != dtype) { rc = SMARTMEM_ERR_SHAPE; break; }
      if (!state_from_desc(w).fresh) { rc = SMARTMEM_ERR_UNSUPPORTED; break; }
      st.weight = wi;
      st.K = w.shape[1];
      st.N = w.shape[0];
      st.M = prod(A.state.shape) / st.K;
      rc = finalize_map(A.state, {0, nd - 1, nd}, esz, &st.map[0], apg);
      st.n_batch_atoms[0] = apg[0];
      st.n_row_atoms[0] = apg[1];
      oshape.assign(A.state.shape.begin(), A.state.shape.end() - 1);
      oshape.push_back(st.N);
    } else if (c.kind == SMARTMEM_OP_BMM_NT) {
      st.kind = STEP_BMM_NT;
      int bi = c.side_input[0];
      if (bi < 1 || bi >= n_inputs) { rc = SMARTMEM_ERR_INVALID_ARG; break; }
      if (nd < 2 || inputs[bi].dtype != dtype) { rc = SMARTMEM_ERR_SHAPE; break; }
      RunResult Bq;
      rc = process_run(p, ops, i, j, inputs[bi], bi, mode, esz, &Bq);
      if (rc != SMARTMEM_OK) break;
      const auto& sa = A.state.shape;
      const auto& sb = Bq.state.shape;
      if (sb.size() != sa.size()) { rc = SMARTMEM_ERR_SHAPE; break; }
      for (int k = 0; k < nd; ++k)
        if (k != nd - 2 && sa[k] != sb[k]) rc = SMARTMEM_ERR_SHAPE;
      if (rc != SMARTMEM_OK) break;
      st.src[1] = Bq.src;
      st.seq[1] = Bq.seq;
      st.M = sa[nd - 2];
      st.N = sb[nd - 2];
      st.K = sa[nd - 1];
      st.batch = prod(sa) / (st.M * st.K);
      rc = finalize_map(A.state, {nd - 2, nd - 1, nd}, esz, &st.map[0], apg);
      st.n_batch_atoms[0] = apg[0];
      st.n_row_atoms[0] = apg[1];
      if (rc == SMARTMEM_OK) rc = finalize_map(Bq.state, {nd - 2, nd - 1, nd}, esz, &st.map[1], apg);
      st.n_batch_atoms[1] = apg[0];
      st.n_row_atoms[1] = apg[1];
      oshape.assign(sa.begin(), sa.end() - 1);
      oshape.push_back(st.N);
    } else if (c.kind == SMARTMEM_OP_LAYERNORM) {
      st.kind = STEP_NORM;
      const int gi = c.side_input[0], bi = c.side_input[1];
      if (gi < 1 || gi >= n_inputs || bi < 1 || bi >= n_inputs) { rc = SMARTMEM_ERR_INVALID_ARG; break; }
      if (nd < 1 || !(c.eps > 0.f)) { rc = SMARTMEM_ERR_INVALID_ARG; break; }
      const int64_t C = A.state.shape[nd - 1];
      for (int wi : {gi, bi}) {
        const smartmem_tensor_desc_t& w = inputs[wi];
        if (w.ndim != 1 || w.shape[0] != C || w.dtype != dtype) rc = SMARTMEM_ERR_SHAPE;
        else if (!state_from_desc(w).fresh) rc = SMARTMEM_ERR_UNSUPPORTED;
      }
      if (rc != SMARTMEM_OK) break;
      st.weight = gi;
      st.weight2 = bi;
      st.eps = c.eps;
      st.K = C;
      st.M = prod(A.state.shape) / C;
      rc = finalize_map(A.state, {nd - 1, nd}, esz, &st.map[0], apg);
      if (rc != SMARTMEM_OK) break;
      // the kernel fetches a row as 16-byte vectors through the map: they must not straddle a contiguous run, and
      // a warp holds the row in registers; otherwise the run is materialised first (as EXPLICIT does anyway)
      const int vec = 16 / esz;
      const bool foldable = (st.map[0].klass != 3 && st.map[0].vec_elems % vec == 0 && C % vec == 0 && C / vec <= 128) ||
                            layernorm_strided_form(st.map[0], esz, C);       // or: channels-first producer, tokens contiguous
      if (!foldable && st.map[0].klass != 0) {
        Step cp;
        cp.kind = STEP_COPY;
        cp.dtype = dtype;
        cp.is_layout_copy = true;
        cp.src[0] = A.src;
        int apg1[1];
        rc = finalize_map(A.state, {nd}, esz, &cp.map[0], apg1);
        if (rc != SMARTMEM_OK) break;
        cp.seq[0] = A.seq;
        cp.dst = new_slot(p, cp.map[0].n_elements, esz);
        p->steps.push_back(cp);
        const smartmem_tensor_desc_t ndsc = contiguous_desc(A.state.shape, dtype);
        TState fresh = state_from_desc(ndsc);
        st.src[0] = cp.dst;
        st.seq[0] = seq_from_desc(ndsc);
        rc = finalize_map(fresh, {nd - 1, nd}, esz, &st.map[0], apg);
        if (rc != SMARTMEM_OK) break;
      }
      oshape = A.state.shape;
    } else {
      rc = SMARTMEM_ERR_INVALID_ARG;
    }
    if (rc != SMARTMEM_OK) break;
    st.dst = last ? -1 : new_slot(p, prod(oshape), esz);
    p->steps.push_back(st);
    cur = contiguous_desc(oshape, dtype);
    cur_src = st.dst;
    i = j + 1;
  }
  if (rc != SMARTMEM_OK) {
    delete p;
    return rc;
  }
  p->out_desc = cur;
  size_t off = 0;
  for (size_t b : p->slot_bytes) {
    p->slot_offset.push_back(off);
    off += b;
  }
  p->workspace_bytes = off;
  *out_plan = p;
  return SMARTMEM_OK;
}

int smartmem_plan_destroy(smartmem_plan_t* plan) {
  delete plan;
  return SMARTMEM_OK;
}

int smartmem_plan_num_steps(const smartmem_plan_t* plan, int32_t* n_steps, int32_t* n_copies) {
  if (!plan || !n_steps || !n_copies) return SMARTMEM_ERR_INVALID_ARG;
  *n_steps = (int)plan->steps.size();
  *n_copies = 0;
  for (auto& s : plan->steps) *n_copies += s.is_layout_copy ? 1 : 0;
  return SMARTMEM_OK;
}

int smartmem_plan_get_map(const smartmem_plan_t* plan, int32_t step, int32_t operand, smartmem_index_map_t* out) {
  if (!plan || !out || step < 0 || step >= (int)plan->steps.size() || operand < 0 || operand > 1)
    return SMARTMEM_ERR_INVALID_ARG;
  if (operand == 1 && plan->steps[step].kind != STEP_BMM_NT) return SMARTMEM_ERR_INVALID_ARG;
  *out = plan->steps[step].map[operand];
  return SMARTMEM_OK;
}

int smartmem_plan_output_desc(const smartmem_plan_t* plan, smartmem_tensor_desc_t* out) {
  if (!plan || !out) return SMARTMEM_ERR_INVALID_ARG;
  *out = plan->out_desc;
  return SMARTMEM_OK;
}

int smartmem_plan_workspace_bytes(const smartmem_plan_t* plan, size_t* bytes) {
  if (!plan || !bytes) return SMARTMEM_ERR_INVALID_ARG;
  *bytes = plan->workspace_bytes;
  return SMARTMEM_OK;
}

int64_t smartmem_map_eval(const smartmem_index_map_t* m, int64_t idx) {
  if (!m || m->klass == 3 || idx < 0 || idx >= m->n_elements) return -1;
  int64_t off = m->base;
  int64_t u[SMARTMEM_MAX_ROLLS] = {0, 0, 0, 0};
  for (int a = m->n_atoms - 1; a >= 0; --a) {
    int64_t digit = idx % m->extent[a];
    idx /= m->extent[a];
    if (m->roll_of[a] < 0) off += digit * m->src_stride[a];
    else u[m->roll_of[a]] += digit * m->roll_weight[a];
  }
  for (int r = 0; r < m->n_rolls; ++r) {
    int64_t v = (u[r] + m->roll_shift[r]) % m->roll_mod[r];
    for (int k = m->roll_n_parts[r] - 1; k >= 0; --k) {
      off += (v % m->roll_part_extent[r][k]) * m->roll_part_stride[r][k];
      v /= m->roll_part_extent[r][k];
    }
  }
  return off;
}

int64_t smartmem_plan_eval_sequential(const smartmem_plan_t* plan, int32_t step, int32_t operand, int64_t idx) {
  if (!plan || step < 0 || step >= (int)plan->steps.size() || operand < 0 || operand > 1) return -1;
  const Step& s = plan->steps[step];
  if (idx < 0 || idx >= s.map[operand].n_elements) return -1;
  return s.seq[operand].eval(idx);
}

const char* smartmem_status_string(int32_t s) {
  switch (s) {
    case SMARTMEM_OK: return "ok";
    case SMARTMEM_ERR_INVALID_ARG: return "invalid argument";
    case SMARTMEM_ERR_SHAPE: return "shape mismatch";
    case SMARTMEM_ERR_UNSUPPORTED: return "unsupported";
    case SMARTMEM_ERR_WORKSPACE: return "workspace too small";
    case SMARTMEM_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
    case SMARTMEM_ERR_CUDA: return "CUDA error or no device";
    case SMARTMEM_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

}  // extern "C"
