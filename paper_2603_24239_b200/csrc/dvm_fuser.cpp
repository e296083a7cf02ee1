// The streaming runtime operator fuser (Sec. 5.2, dynamic computation graphs): host-side only.  It talks to
// the rest of the library through the public C ABI (dvm_program_*, dvm_encode, dvm_launch, dvm_launch_stacked).
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <vector>

#include "../../include/dvm.h"
#include "../../include/dvm_fuser.h"

namespace {

enum OpKind { OP_UNARY, OP_BINARY, OP_SCALAR, OP_REDUCE, OP_COMPARE, OP_SELECT, OP_CAST, OP_MATMUL };

struct FValue {
  int dtype;
  dvm_shape shape;
  void* ptr;
  int op;         // index into `ops` of the pending operator that produces it, or -1: it lies in memory
  bool released;  // the framework holds no reference any more
  bool valid;     // false: released and never stored
};

struct FOp {
  int kind, op, x, y;  // (OP_SELECT: x the condition, y the then-value; OP_CAST: op the target type)
  float s;
  int out;    // value id of the result
  int group;  // index into `groups`
  int z;      // OP_SELECT: the else-value, otherwise -1
};

// the value operands of an operator: x, then y and z where the kind has them (-1 otherwise)
inline void operands_of(const FOp& o, int v[3]) {
  v[0] = o.x;
  v[1] = (o.kind == OP_BINARY || o.kind == OP_COMPARE || o.kind == OP_SELECT || o.kind == OP_MATMUL) ? o.y : -1;
  v[2] = o.kind == OP_SELECT ? o.z : -1;
}

struct FGroup {
  std::vector<int> ops;  // pending operator indices, in arrival order
  int level;             // 0: reads only tensors in memory; else 1 + the deepest group it reads from
  bool alive;            // false: merged into another group
};

struct Built {  // one group as an operator program
  dvm_program* prog = nullptr;
  std::vector<int> inputs;   // value ids, in program input order
  std::vector<int> outputs;  // value ids, in program output order
};

}  // namespace

struct dvm_fuser {
  void* stream;
  std::vector<FValue> values;
  std::vector<FOp> ops;
  std::vector<FGroup> groups;
  int64_t n_ops = 0, n_groups = 0, n_launches = 0, n_elided = 0;
  bool temporal = true;  // dependent groups share one launch (dvm_launch_stacked_levels)
};

namespace {

// Levels of more tiles than this run as launches of their own (a tile is 256 threads x 16 elements here).
constexpr int64_t kTemporalMaxTilesPerLevel = 1024;

bool value_ok(const dvm_fuser* f, int v) { return v >= 0 && v < (int)f->values.size() && f->values[v].valid; }

// Does another group than `g` read value v (among the pending operators)?
bool read_elsewhere(const dvm_fuser* f, int v, int g) {
  for (const FOp& o : f->ops) {
    if (o.group == g) continue;
    int xs[3];
    operands_of(o, xs);
    if (xs[0] == v || xs[1] == v || xs[2] == v) return true;
  }
  return false;
}

// Builds the operator program of a group made of `op_list` (pending operator indices in arrival order,
// possibly with `extra` -- an operator not yet in f->ops -- at the end).  for_decision: every value that
// is not released counts as an output (later operators are unknown yet).
int build(const dvm_fuser* f, const std::vector<int>& op_list, const FOp* extra, int group, bool for_decision, Built* b) {
  int st = dvm_program_create(&b->prog);
  if (st != DVM_OK) return st;
  std::vector<std::pair<int, int>> ids;  // value id -> program value id
  auto find = [&](int v) {
    for (auto& p : ids)
      if (p.first == v) return p.second;
    return -1;
  };
  auto operand = [&](int v, int* pid) -> int {
    *pid = find(v);
    if (*pid >= 0) return DVM_OK;
    const FValue& val = f->values[v];
    int s2 = dvm_program_input(b->prog, val.dtype, val.shape.rank, pid);
    if (s2 == DVM_OK) {
      ids.push_back({v, *pid});
      b->inputs.push_back(v);
    }
    return s2;
  };
  const size_t n = op_list.size() + (extra ? 1 : 0);
  std::vector<const FOp*> seq;
  for (int k : op_list) seq.push_back(&f->ops[k]);
  if (extra) seq.push_back(extra);
  for (size_t k = 0; k < n && st == DVM_OK; ++k) {
    const FOp& o = *seq[k];
    int px = -1, py = -1, pz = -1, pid = -1;
    int xs[3];
    operands_of(o, xs);
    st = operand(xs[0], &px);
    if (st == DVM_OK && xs[1] >= 0) st = operand(xs[1], &py);
    if (st == DVM_OK && xs[2] >= 0) st = operand(xs[2], &pz);
    if (st != DVM_OK) break;
    switch (o.kind) {
      case OP_UNARY: st = dvm_program_unary(b->prog, o.op, px, &pid); break;
      case OP_BINARY: st = dvm_program_binary(b->prog, o.op, px, py, &pid); break;
      case OP_SCALAR: st = dvm_program_scalar(b->prog, o.op, px, o.s, &pid); break;
      case OP_COMPARE: st = dvm_program_compare(b->prog, o.op, px, py, &pid); break;
      case OP_SELECT: st = dvm_program_select(b->prog, px, py, pz, &pid); break;
      case OP_CAST: st = dvm_program_cast(b->prog, px, o.op, &pid); break;
      case OP_MATMUL: st = dvm_program_matmul(b->prog, px, py, &pid); break;
      default: st = dvm_program_reduce(b->prog, o.op, px, o.y, &pid); break;  // (OP_REDUCE: y is the axis)
    }
    if (st == DVM_OK) ids.push_back({o.out, pid});
  }
  for (size_t k = 0; k < n && st == DVM_OK; ++k) {
    const FOp& o = *seq[k];
    const FValue& val = f->values[o.out];
    const bool is_extra = extra && seq[k] == extra;
    const bool store = for_decision ? (!val.released || is_extra) : (!val.released || read_elsewhere(f, o.out, group));
    if (!store) continue;
    st = dvm_program_output(b->prog, find(o.out), val.dtype);
    if (st == DVM_OK) b->outputs.push_back(o.out);
  }
  if (st == DVM_OK && b->outputs.empty()) st = DVM_ERR_INVALID_ARG;  // callers skip groups with nothing to store
  if (st == DVM_OK) st = dvm_program_finalize(b->prog);
  if (st != DVM_OK) {
    dvm_program_destroy(b->prog);
    b->prog = nullptr;
  }
  return st;
}

// Encodes a built group for its concrete input shapes; out_shapes (optional) in program output order.
int encode(const dvm_fuser* f, const Built& b, std::vector<uint64_t>* code, size_t* size, std::vector<dvm_shape>* out_shapes) {
  std::vector<dvm_shape> in;
  for (int v : b.inputs) in.push_back(f->values[v].shape);
  const size_t cap = dvm_code_max_size(b.prog);
  code->assign((cap + 7) / 8, 0);
  std::vector<dvm_shape> os(b.outputs.size());
  int st = dvm_encode(b.prog, in.data(), (int)in.size(), nullptr, 0, code->data(), cap, size, os.data(), (int)os.size());
  if (st == DVM_OK && out_shapes) *out_shapes = os;
  return st;
}

int add_op(dvm_fuser* f, FOp o, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value) {
  if (!f || !value || !out_ptr || out_dtype < DVM_F32 || out_dtype > DVM_I32) return DVM_ERR_INVALID_ARG;
  int xs[3];
  operands_of(o, xs);
  for (int k = 0; k < 3; ++k)
    if ((k == 0 || xs[k] >= 0) && !value_ok(f, xs[k])) return DVM_ERR_INVALID_ARG;
  if ((int)f->ops.size() >= DVM_FUSER_MAX_OPS) {  // flush condition: the operator buffer is full
    int st = dvm_fuser_flush(f);
    if (st != DVM_OK) return st;
  }
  // the result value (its shape comes from the trial encode below)
  FValue nv = {};
  nv.dtype = out_dtype;
  nv.ptr = out_ptr;
  nv.op = (int)f->ops.size();
  nv.released = false;
  nv.valid = true;
  f->values.push_back(nv);
  o.out = (int)f->values.size() - 1;

  // producer groups of the operands
  int prod[3] = {-1, -1, -1}, np = 0;
  for (int k = 0; k < 3; ++k)
    if (xs[k] >= 0 && f->values[xs[k]].op >= 0) {
      const int g = f->ops[f->values[xs[k]].op].group;
      bool seen = false;
      for (int q = 0; q < np; ++q) seen = seen || prod[q] == g;
      if (!seen) prod[np++] = g;
    }
  // candidate: the operator joins the producers' group (two producer groups: they merge around it)
  int joined = -1, st = DVM_OK;
  std::vector<dvm_shape> shapes;
  // two producer groups merge around the operator only when both read nothing but tensors in memory:
  // then no third group can sit between them, and the merged group cannot end up depending on itself
  bool can_join = np == 1;
  if (np >= 2) {
    can_join = true;
    for (int q = 0; q < np; ++q) can_join = can_join && f->groups[prod[q]].level == 0;
  }
  if (can_join) {
    std::vector<int> cand = f->groups[prod[0]].ops;
    for (int q = 1; q < np; ++q) cand.insert(cand.end(), f->groups[prod[q]].ops.begin(), f->groups[prod[q]].ops.end());
    if (np >= 2) std::sort(cand.begin(), cand.end());
    Built b;
    st = build(f, cand, &o, prod[0], true, &b);
    if (st == DVM_OK) {
      std::vector<uint64_t> code;
      size_t size = 0;
      st = encode(f, b, &code, &size, &shapes);
      if (st == DVM_OK) {  // the iterations merge: pattern-based fusion
        joined = prod[0];
        for (size_t k = 0; k < b.outputs.size(); ++k)
          if (b.outputs[k] == o.out) f->values[o.out].shape = shapes[k];
      }
      dvm_program_destroy(b.prog);
    }
  }
  if (joined >= 0) {
    for (int q = 1; q < np; ++q) {  // merge the other producer groups into the first
      FGroup& a = f->groups[prod[0]];
      FGroup& c = f->groups[prod[q]];
      for (int k : c.ops) f->ops[k].group = prod[0];
      a.ops.insert(a.ops.end(), c.ops.begin(), c.ops.end());
      std::sort(a.ops.begin(), a.ops.end());
      a.level = std::max(a.level, c.level);
      c.ops.clear();
      c.alive = false;
    }
    o.group = joined;
    f->groups[joined].ops.push_back((int)f->ops.size());
  } else {
    // a group of its own: it must at least encode alone
    Built b;
    st = build(f, {}, &o, -1, true, &b);
    std::vector<uint64_t> code;
    size_t size = 0;
    if (st == DVM_OK) {
      st = encode(f, b, &code, &size, &shapes);
      dvm_program_destroy(b.prog);
    }
    if (st != DVM_OK) {
      f->values.pop_back();
      return st;
    }
    f->values[o.out].shape = shapes[0];
    FGroup g;
    g.alive = true;
    g.level = 0;
    for (int k = 0; k < np; ++k) g.level = std::max(g.level, f->groups[prod[k]].level + 1);
    g.ops.push_back((int)f->ops.size());
    f->groups.push_back(g);
    o.group = (int)f->groups.size() - 1;
  }
  f->ops.push_back(o);
  f->n_ops++;
  if (out_shape) *out_shape = f->values[o.out].shape;
  *value = o.out;
  return DVM_OK;
}

}  // namespace

extern "C" int dvm_fuser_create(dvm_fuser** out, void* cuda_stream) {
  if (!out) return DVM_ERR_INVALID_ARG;
  *out = new (std::nothrow) dvm_fuser();
  if (!*out) return DVM_ERR_INVALID_ARG;
  (*out)->stream = cuda_stream;
  return DVM_OK;
}

extern "C" void dvm_fuser_destroy(dvm_fuser* f) { delete f; }

extern "C" int dvm_fuser_tensor(dvm_fuser* f, int dtype, const dvm_shape* shape, void* device_ptr, int* value) {
  if (!f || !shape || !device_ptr || !value || (dtype != DVM_F32 && dtype != DVM_BF16)) return DVM_ERR_INVALID_ARG;
  if (shape->rank < 0 || shape->rank > DVM_MAX_RANK) return DVM_ERR_INVALID_ARG;
  FValue v = {};
  v.dtype = dtype;
  v.shape = *shape;
  v.ptr = device_ptr;
  v.op = -1;
  v.released = false;
  v.valid = true;
  f->values.push_back(v);
  *value = (int)f->values.size() - 1;
  return DVM_OK;
}

extern "C" int dvm_fuser_unary(dvm_fuser* f, int op, int x, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value) {
  FOp o = {OP_UNARY, op, x, -1, 0.f, -1, -1, -1};
  return add_op(f, o, out_dtype, out_ptr, out_shape, value);
}
extern "C" int dvm_fuser_binary(dvm_fuser* f, int op, int x, int y, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value) {
  FOp o = {OP_BINARY, op, x, y, 0.f, -1, -1, -1};
  return add_op(f, o, out_dtype, out_ptr, out_shape, value);
}
extern "C" int dvm_fuser_scalar(dvm_fuser* f, int op, int x, float s, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value) {
  FOp o = {OP_SCALAR, op, x, -1, s, -1, -1, -1};
  return add_op(f, o, out_dtype, out_ptr, out_shape, value);
}
extern "C" int dvm_fuser_reduce(dvm_fuser* f, int op, int x, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value) {
  FOp o = {OP_REDUCE, op, x, -1, 0.f, -1, -1, -1};
  return add_op(f, o, out_dtype, out_ptr, out_shape, value);
}
extern "C" int dvm_fuser_reduce_axis(dvm_fuser* f, int op, int x, int axis, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value) {
  if (axis >= 0) return DVM_ERR_INVALID_ARG;  // counted from the end, like dvm_program_reduce
  FOp o = {OP_REDUCE, op, x, axis, 0.f, -1, -1, -1};
  return add_op(f, o, out_dtype, out_ptr, out_shape, value);
}
extern "C" int dvm_fuser_compare(dvm_fuser* f, int op, int x, int y, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value) {
  FOp o = {OP_COMPARE, op, x, y, 0.f, -1, -1, -1};
  return add_op(f, o, out_dtype, out_ptr, out_shape, value);
}
extern "C" int dvm_fuser_select(dvm_fuser* f, int cond, int x, int y, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value) {
  FOp o = {OP_SELECT, 0, cond, x, 0.f, -1, -1, y};
  return add_op(f, o, out_dtype, out_ptr, out_shape, value);
}
extern "C" int dvm_fuser_cast(dvm_fuser* f, int x, int dtype, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value) {
  FOp o = {OP_CAST, dtype, x, -1, 0.f, -1, -1, -1};
  return add_op(f, o, out_dtype, out_ptr, out_shape, value);
}
extern "C" int dvm_fuser_matmul(dvm_fuser* f, int a, int b, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value) {
  FOp o = {OP_MATMUL, 0, a, b, 0.f, -1, -1, -1};
  return add_op(f, o, out_dtype, out_ptr, out_shape, value);
}

extern "C" int dvm_fuser_release(dvm_fuser* f, int value) {
  if (!f || value < 0 || value >= (int)f->values.size()) return DVM_ERR_INVALID_ARG;
  f->values[value].released = true;
  return DVM_OK;
}

extern "C" int dvm_fuser_pending(const dvm_fuser* f, int* n_ops, int* n_groups) {
  if (!f) return DVM_ERR_INVALID_ARG;
  if (n_ops) *n_ops = (int)f->ops.size();
  if (n_groups) {
    int g = 0;
    for (const FGroup& gr : f->groups) g += gr.alive ? 1 : 0;
    *n_groups = g;
  }
  return DVM_OK;
}

extern "C" int dvm_fuser_stats(const dvm_fuser* f, int64_t* n_ops, int64_t* n_groups, int64_t* n_launches, int64_t* n_stores_elided) {
  if (!f) return DVM_ERR_INVALID_ARG;
  if (n_ops) *n_ops = f->n_ops;
  if (n_groups) *n_groups = f->n_groups;
  if (n_launches) *n_launches = f->n_launches;
  if (n_stores_elided) *n_stores_elided = f->n_elided;
  return DVM_OK;
}

extern "C" int dvm_fuser_set_temporal_stacking(dvm_fuser* f, int enabled) {
  if (!f) return DVM_ERR_INVALID_ARG;
  f->temporal = enabled != 0;
  return DVM_OK;
}

extern "C" int dvm_fuser_flush(dvm_fuser* f) {
  if (!f) return DVM_ERR_INVALID_ARG;
  int status = DVM_OK;
  // levels from the dependencies as they stand now: 0 = reads only memory, else 1 + the deepest producer group
  for (FGroup& g : f->groups) g.level = 0;
  for (bool changed = true; changed;) {
    changed = false;
    for (const FOp& o : f->ops) {
      int xs[3];
      operands_of(o, xs);
      for (int k = 0; k < 3; ++k) {
        if (xs[k] < 0 || f->values[xs[k]].op < 0) continue;
        const int h = f->ops[f->values[xs[k]].op].group;
        if (h != o.group && f->groups[o.group].level < f->groups[h].level + 1) {
          f->groups[o.group].level = f->groups[h].level + 1;
          changed = true;
        }
      }
    }
  }
  int max_level = -1;
  for (const FGroup& g : f->groups)
    if (g.alive) max_level = std::max(max_level, g.level);
  // Encode every live group, in level order.  More than one group means a stacked launch, whose programs
  // share one elements-per-thread setting.
  struct Ready {
    std::vector<uint64_t> code;
    size_t size;
    std::vector<void*> tensors;
    int level;
    int64_t tiles;
  };
  std::vector<Ready> ready;
  std::vector<int> order;
  for (int level = 0; level <= max_level; ++level)
    for (int g = 0; g < (int)f->groups.size(); ++g)
      if (f->groups[g].alive && f->groups[g].level == level) order.push_back(g);
  const int saved_v = dvm_get_elems_per_thread();
  const bool stacked = order.size() > 1;
  const int saved_ctas = dvm_get_min_resident_ctas();
  if (stacked) {
    dvm_set_elems_per_thread(16);
    dvm_set_min_resident_ctas(2);  // the launch's CTAs are sized by its largest program
  }
  for (int g : order) {
    Built b;
    int st = build(f, f->groups[g].ops, nullptr, g, false, &b);
    if (st == DVM_ERR_INVALID_ARG && !b.prog) {
      // nothing of this group is needed any more (every result released and unread): dead code
      bool none = true;
      for (int k : f->groups[g].ops)
        if (!f->values[f->ops[k].out].released || read_elsewhere(f, f->ops[k].out, g)) none = false;
      if (none) {
        f->n_elided += (int64_t)f->groups[g].ops.size();
        continue;
      }
    }
    if (st != DVM_OK) { status = st; break; }
    Ready r;
    r.level = f->groups[g].level;
    r.tiles = 0;
    st = encode(f, b, &r.code, &r.size, nullptr);
    if (st == DVM_OK) st = dvm_code_info(r.code.data(), r.size, nullptr, &r.tiles, nullptr, nullptr, nullptr, nullptr);
    if (st == DVM_OK) {
      for (int v : b.inputs) r.tensors.push_back(f->values[v].ptr);
      for (int v : b.outputs) r.tensors.push_back(f->values[v].ptr);
      f->n_elided += (int64_t)f->groups[g].ops.size() - (int64_t)b.outputs.size();
      f->n_groups++;
      ready.push_back(std::move(r));
    }
    dvm_program_destroy(b.prog);
    if (st != DVM_OK) { status = st; break; }
  }
  if (stacked) {
    dvm_set_elems_per_thread(saved_v);
    dvm_set_min_resident_ctas(saved_ctas);
  }

  // Launch programs [lo, hi) of `ready`: one stacked kernel (with in-kernel level waits when they span
  // several levels), or one launch each when they do not fit one parameter block.
  auto launch_range = [&](size_t lo, size_t hi) -> int {
    if (hi - lo == 1) {
      int st = dvm_launch(ready[lo].code.data(), ready[lo].size, ready[lo].tensors.data(), (int)ready[lo].tensors.size(), f->stream);
      if (st == DVM_OK) f->n_launches++;
      return st;
    }
    std::vector<const void*> codes;
    std::vector<size_t> sizes;
    std::vector<void* const*> tls;
    std::vector<int> nts, levels;
    for (size_t k = lo; k < hi; ++k) {
      codes.push_back(ready[k].code.data());
      sizes.push_back(ready[k].size);
      tls.push_back(ready[k].tensors.data());
      nts.push_back((int)ready[k].tensors.size());
      levels.push_back(ready[k].level);
    }
    int st;
    if (levels.front() != levels.back())  // temporal stacking of dependent groups (Sec. 5.1)
      st = dvm_launch_stacked_levels((int)(hi - lo), codes.data(), sizes.data(), tls.data(), nts.data(), levels.data(), f->stream);
    else  // the groups of one level do not depend on one another: spatial stacking (Sec. 5.1)
      st = dvm_launch_stacked((int)(hi - lo), codes.data(), sizes.data(), tls.data(), nts.data(), f->stream);
    if (st == DVM_OK) f->n_launches++;
    return st;
  };
  // One kernel for all levels pays while the levels are short: an in-kernel level change costs a few
  // microseconds of drained pipeline, about what a kernel boundary costs on the device, but it saves the host
  // one launch per level; with long levels the host is far ahead of the device anyway, and a level that is
  // alone in its launch runs the one-program interpreter variant, which is the faster one per tile.
  bool short_levels = true;
  for (size_t lo = 0; lo < ready.size();) {
    size_t hi = lo;
    int64_t tiles = 0;
    for (; hi < ready.size() && ready[hi].level == ready[lo].level; ++hi) tiles += ready[hi].tiles;
    if (tiles > kTemporalMaxTilesPerLevel) short_levels = false;
    lo = hi;
  }
  if (status == DVM_OK && !ready.empty()) {
    int st = (f->temporal && short_levels) ? launch_range(0, ready.size()) : DVM_ERR_TOO_LARGE;
    if (st == DVM_ERR_TOO_LARGE || st == DVM_ERR_UNSUPPORTED) {
      // one launch per level, in order on the stream
      st = DVM_OK;
      for (size_t lo = 0; lo < ready.size() && st == DVM_OK;) {
        size_t hi = lo;
        while (hi < ready.size() && ready[hi].level == ready[lo].level) ++hi;
        st = launch_range(lo, hi);
        if (st == DVM_ERR_TOO_LARGE || st == DVM_ERR_UNSUPPORTED) {
          st = DVM_OK;  // too many / too large for one parameter block: one launch each
          for (size_t k = lo; k < hi && st == DVM_OK; ++k) st = launch_range(k, k + 1);
        }
        lo = hi;
      }
    }
    status = st;
  }
  // everything pending has been issued (or failed): results now lie in memory, unless they were never stored
  for (const FOp& o : f->ops) {
    FValue& v = f->values[o.out];
    if (v.released && !read_elsewhere(f, o.out, o.group)) v.valid = false;
    v.op = -1;
  }
  f->ops.clear();
  f->groups.clear();
  return status;
}
