// Host half of the operator compiler: program description, per-instance shape
// inference, shape tiling, bytecode encoding, verification and the readable dump.
// No CUDA here; dvm_encode performs no heap allocation.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <chrono>

#include <utility>

#include "../../include/dvm.h"
#include "dvm_format.h"
#include "dvm_internal.h"
#include "dvm_program.h"

// ---------------------------------------------------------------------------
// Program description
// ---------------------------------------------------------------------------
static thread_local int g_num_cores = 0;
static const int kDefaultCores = 148 * 3;

static thread_local int g_elems_per_thread = 0;
extern "C" void dvm_set_elems_per_thread(int v) { g_elems_per_thread = (v == 16 || v == 24 || v == 32) ? v : 0; }
extern "C" int dvm_get_elems_per_thread(void) { return g_elems_per_thread; }
static thread_local int g_min_resident_ctas = 0;
static thread_local bool g_stack_one_slot = false;  // (n = 3: two CTAs per SM that hold ONE tile slot each)
extern "C" void dvm_set_min_resident_ctas(int n) {
  g_min_resident_ctas = (n == 2 || n == 3) ? 2 : 0;
  g_stack_one_slot = n == 3;
}
extern "C" int dvm_get_min_resident_ctas(void) { return g_stack_one_slot ? 3 : g_min_resident_ctas; }
extern "C" void dvm_set_num_cores(int n) { g_num_cores = n > 0 ? n : 0; }
extern "C" int dvm_get_num_cores(void) { return g_num_cores > 0 ? g_num_cores : kDefaultCores; }

extern "C" int dvm_program_create(dvm_program** out) {
  if (!out) return DVM_ERR_INVALID_ARG;
  dvm_program* p = (dvm_program*)calloc(1, sizeof(dvm_program));
  if (!p) return DVM_ERR_INVALID_ARG;
  *out = p;
  return DVM_OK;
}

extern "C" void dvm_program_destroy(dvm_program* p) { free(p); }

static int push_node(dvm_program* p, const Node& n, int* value_id) {
  if (!p || !value_id) return DVM_ERR_INVALID_ARG;
  if (p->finalized) return DVM_ERR_INVALID_ARG;
  if (p->n_nodes >= DVM_MAX_NODES) return DVM_ERR_TOO_LARGE;
  p->nodes[p->n_nodes] = n;
  *value_id = p->n_nodes++;
  return DVM_OK;
}

static bool valid_value(const dvm_program* p, int v) { return p && v >= 0 && v < p->n_nodes; }

extern "C" int dvm_program_input(dvm_program* p, int dtype, int rank, int* value_id) {
  if (!p) return DVM_ERR_INVALID_ARG;
  if (dtype != DVM_F32 && dtype != DVM_BF16) return DVM_ERR_INVALID_ARG;
  if (rank < 0 || rank > DVM_MAX_RANK) return DVM_ERR_INVALID_ARG;
  if (p->n_inputs >= DVM_MAX_TENSORS) return DVM_ERR_TOO_LARGE;
  Node n = {};
  n.kind = NK_INPUT;
  n.dtype = (uint8_t)dtype;
  n.rank = (int8_t)rank;
  n.x = n.y = n.param = -1;
  int st = push_node(p, n, value_id);
  if (st == DVM_OK) p->inputs[p->n_inputs++] = (int16_t)*value_id;
  return st;
}

extern "C" int dvm_program_unary(dvm_program* p, int op, int x, int* value_id) {
  if (!valid_value(p, x) || op < 0 || op > DVM_ISFINITE) return DVM_ERR_INVALID_ARG;
  Node n = {};
  n.kind = NK_UNARY;
  n.op = (uint8_t)op;
  n.x = (int16_t)x;
  n.y = n.param = -1;
  return push_node(p, n, value_id);
}

extern "C" int dvm_program_binary(dvm_program* p, int op, int x, int y, int* value_id) {
  if (!valid_value(p, x) || !valid_value(p, y) || op < 0 || op > DVM_POW) return DVM_ERR_INVALID_ARG;
  Node n = {};
  // Pow shares the two-tile-operand instruction class of the comparisons (extended interpreter variant)
  n.kind = op == DVM_POW ? NK_COMPARE : NK_BINARY;
  n.op = (uint8_t)(op == DVM_POW ? DVM_C_POW : op);
  n.x = (int16_t)x;
  n.y = (int16_t)y;
  n.param = -1;
  return push_node(p, n, value_id);
}

extern "C" int dvm_program_scalar(dvm_program* p, int op, int x, float s, int* value_id) {
  if (!valid_value(p, x) || op < 0 || op > DVM_MULS) return DVM_ERR_INVALID_ARG;
  Node n = {};
  n.kind = NK_SCALAR;
  n.op = (uint8_t)op;
  n.x = (int16_t)x;
  n.y = n.param = -1;
  n.imm = s;
  return push_node(p, n, value_id);
}

extern "C" int dvm_program_scalar_param(dvm_program* p, int op, int x, int param, int* value_id) {
  if (!valid_value(p, x) || op < 0 || op > DVM_MULS || param < 0 || param >= 64)
    return DVM_ERR_INVALID_ARG;
  Node n = {};
  n.kind = NK_SCALAR;
  n.op = (uint8_t)op;
  n.x = (int16_t)x;
  n.y = -1;
  n.param = (int16_t)param;
  int st = push_node(p, n, value_id);
  if (st == DVM_OK && param + 1 > p->n_params) p->n_params = param + 1;
  return st;
}

extern "C" int dvm_program_cast(dvm_program* p, int x, int dtype, int* value_id) {
  if (!valid_value(p, x) || dtype < DVM_F32 || dtype > DVM_I32) return DVM_ERR_INVALID_ARG;
  Node n = {};
  n.kind = NK_CAST;
  n.dtype = (uint8_t)dtype;
  n.x = (int16_t)x;
  n.y = n.param = -1;
  return push_node(p, n, value_id);
}

extern "C" int dvm_program_reduce(dvm_program* p, int op, int x, int axis, int* value_id) {
  if (!valid_value(p, x) || op < 0 || op > DVM_RMIN) return DVM_ERR_INVALID_ARG;
  if (axis > -1 || axis < -DVM_MAX_RANK) return DVM_ERR_INVALID_ARG;  // the axis counts from the end: -1 .. -DVM_MAX_RANK
  Node n = {};
  n.kind = NK_REDUCE;
  n.op = (uint8_t)op;
  n.x = (int16_t)x;
  n.y = -1;
  n.param = (int16_t)axis;
  return push_node(p, n, value_id);
}

extern "C" int dvm_program_compare(dvm_program* p, int op, int x, int y, int* value_id) {
  if (!valid_value(p, x) || !valid_value(p, y) || op < 0 || op > DVM_CMP_NE) return DVM_ERR_INVALID_ARG;
  Node n = {};
  n.kind = NK_COMPARE;
  n.op = (uint8_t)op;
  n.x = (int16_t)x;
  n.y = (int16_t)y;
  n.param = -1;
  return push_node(p, n, value_id);
}

extern "C" int dvm_program_select(dvm_program* p, int cond, int x, int y, int* value_id) {
  if (!valid_value(p, cond) || !valid_value(p, x) || !valid_value(p, y)) return DVM_ERR_INVALID_ARG;
  Node n = {};
  n.kind = NK_SELECT;
  n.x = (int16_t)cond;
  n.y = (int16_t)x;
  n.param = (int16_t)y;
  return push_node(p, n, value_id);
}

extern "C" int dvm_program_matmul(dvm_program* p, int a, int b, int* value_id) {
  if (!valid_value(p, a) || !valid_value(p, b)) return DVM_ERR_INVALID_ARG;
  if (p->nodes[a].kind != NK_INPUT || p->nodes[b].kind != NK_INPUT) return DVM_ERR_UNSUPPORTED;
  Node n = {};
  n.kind = NK_MATMUL;
  n.x = (int16_t)a;
  n.y = (int16_t)b;
  n.param = -1;
  int st = push_node(p, n, value_id);
  if (st == DVM_OK) p->n_matmul++;
  return st;
}

extern "C" int dvm_program_output(dvm_program* p, int x, int dtype) {
  if (!valid_value(p, x) || dtype < DVM_F32 || dtype > DVM_I32) return DVM_ERR_INVALID_ARG;
  if (p->finalized) return DVM_ERR_INVALID_ARG;
  if (p->n_outputs >= DVM_MAX_TENSORS) return DVM_ERR_TOO_LARGE;
  p->outputs[p->n_outputs].value = (int16_t)x;
  p->outputs[p->n_outputs].dtype = (uint8_t)dtype;
  p->n_outputs++;
  return DVM_OK;
}

extern "C" int dvm_program_finalize(dvm_program* p) {
  if (!p) return DVM_ERR_INVALID_ARG;
  if (p->n_outputs == 0 || p->n_inputs == 0) return DVM_ERR_INVALID_ARG;
  if (p->n_inputs + p->n_outputs > DVM_MAX_TENSORS) return DVM_ERR_TOO_LARGE;
  for (int i = 0; i < p->n_nodes; ++i) {
    const Node& n = p->nodes[i];
    if (n.kind != NK_INPUT && (n.x < 0 || n.x >= i)) return DVM_ERR_INVALID_ARG;
    if ((n.kind == NK_BINARY || n.kind == NK_MATMUL || n.kind == NK_COMPARE || n.kind == NK_SELECT) && (n.y < 0 || n.y >= i))
      return DVM_ERR_INVALID_ARG;
    if (n.kind == NK_SELECT && (n.param < 0 || n.param >= i)) return DVM_ERR_INVALID_ARG;
  }
  if (p->n_matmul > 0) {
    if (p->n_matmul > 2) return DVM_ERR_UNSUPPORTED;
    int a = -1;
    for (int i = 0; i < p->n_nodes; ++i) {
      const Node& n = p->nodes[i];
      if (n.kind == NK_MATMUL) {
        if (a >= 0 && n.x != a) return DVM_ERR_UNSUPPORTED;
        a = n.x;
        if (p->nodes[n.x].dtype != DVM_BF16 || p->nodes[n.y].dtype != DVM_BF16) return DVM_ERR_UNSUPPORTED;
      }
      if (n.kind == NK_REDUCE || n.kind == NK_COMPARE || n.kind == NK_SELECT) return DVM_ERR_UNSUPPORTED;  // epilogues: plain elementwise arithmetic only
      if (n.kind == NK_UNARY && n.op == DVM_ISFINITE) return DVM_ERR_UNSUPPORTED;
    }
  }
  p->finalized = true;
  return DVM_OK;
}

extern "C" int dvm_program_num_inputs(const dvm_program* p) { return p ? p->n_inputs : DVM_ERR_INVALID_ARG; }
extern "C" int dvm_program_num_outputs(const dvm_program* p) { return p ? p->n_outputs : DVM_ERR_INVALID_ARG; }

extern "C" size_t dvm_code_max_size(const dvm_program* p) {
  if (!p) return 0;
  // header + matmul extension + tensor table + operand table + 6 words per node (loads, converts,
  // spills, the operation with immediate) + stores
  size_t words = DVM_HDR_WORDS + DVM_MM_WORDS + 2 * DVM_MAX_TENSORS + DVM_OPD_WORDS * DVM_MAX_OPERANDS +
                 8 * (size_t)p->n_nodes + 4 * (size_t)p->n_outputs + 16;
  return words * 4;
}

// ---------------------------------------------------------------------------
// The paper's tile-size rule and Algorithm 2's tile range (exported for tests)
// ---------------------------------------------------------------------------
static inline int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }

extern "C" int dvm_hardware_align_div(int64_t total, int n_cores, int64_t align, int64_t t_max,
                                      int64_t overhead, int64_t* min_cost_tile, int64_t* rounded_tile,
                                      int64_t* n_tiles, int64_t* tail) {
  if (total <= 0 || n_cores <= 0 || align <= 0 || t_max <= 0 || overhead < 0) return DVM_ERR_INVALID_ARG;
  int64_t hi = total < t_max ? total : t_max;
  int64_t best_t = 1, best_cost = -1;
  for (int64_t t = 1; t <= hi; ++t) {
    int64_t cost = cdiv(cdiv(total, t), n_cores) * (t + overhead);
    if (best_cost < 0 || cost <= best_cost) {  // ties: the larger tile
      best_cost = cost;
      best_t = t;
    }
  }
  int64_t r = cdiv(best_t, align) * align;
  if (r > t_max) r = best_t;  // rounding must respect the tile size limit
  int64_t nt = cdiv(total, best_t);
  if (min_cost_tile) *min_cost_tile = best_t;
  if (rounded_tile) *rounded_tile = r;
  if (n_tiles) *n_tiles = nt;
  if (tail) *tail = total - (nt - 1) * best_t;
  return DVM_OK;
}

extern "C" int dvm_vm_tile_range(int64_t n_tiles, int n_cores, int id, int64_t* begin, int64_t* end) {
  if (n_tiles < 0 || n_cores <= 0 || id < 0 || id >= n_cores || !begin || !end) return DVM_ERR_INVALID_ARG;
  int64_t m = cdiv(n_tiles, n_cores);
  int64_t b = m * id, e = m * (id + 1);
  if (b > n_tiles) b = n_tiles;
  if (e > n_tiles) e = n_tiles;
  *begin = b;
  *end = e;
  return DVM_OK;
}

// ---------------------------------------------------------------------------
// Encode
// ---------------------------------------------------------------------------
namespace {

enum { CLS_TILE = 0, CLS_SCAL = 1 };

struct Operand {       // one global-memory access
  int slot;            // tensor slot
  int dtype;
  int col_stride;      // 1: a tile-class access (it has columns), 0: one value per row
  int64_t cs;          // element stride between the columns of a tile-class access: 1, or what a view gives (ViewLoad / ViewStore)
  int combine;         // output only: 0 plain store, 1 + DVM_SUM / DVM_RMAX / DVM_RMIN: atomic combination (see combine_axis)
  int64_t numel;       // combined output: its elements (the launch pre-fills them with the operation's identity)
  int64_t stride[DVM_MAX_RANK];  // element strides over the dominant dims (before merging)
  int64_t ostride[3];            // after merging: outer dims, innermost first
  bool primary;
};

struct Enc {
  const dvm_program* p;
  int64_t Sd[DVM_MAX_RANK];       // dominant shape
  int64_t dims[DVM_MAX_NODES][DVM_MAX_RANK];  // right-aligned per value
  int8_t cls[DVM_MAX_NODES];
  int16_t alias[DVM_MAX_NODES];   // identity nodes resolve to another value
  // code generation state
  uint32_t loads[4 * DVM_MAX_TENSORS];          // load section
  int n_loads;
  uint32_t body[8 * DVM_MAX_NODES + 64];        // compute section
  int n_body;
  Operand opd[DVM_MAX_OPERANDS];
  int n_opd;
  int16_t uses[DVM_MAX_NODES];
  int8_t lreg_of[DVM_MAX_NODES];  // local (shared-memory) register holding the value, or -1
  int8_t ldt_of[DVM_MAX_NODES];   // element type of that register's content
  int8_t sreg_of[DVM_MAX_NODES];
  int8_t sslot_of[DVM_MAX_NODES]; // local scalar slot of a per-row scalar input
  int16_t tmp_val[DVM_MAX_LREGS]; // temporaries: value held or -1
  int16_t sreg_val[DVM_MAX_SREGS];
  int16_t acc;                    // value in the accumulator or -1
  int n_in_regs, n_tmp_regs, n_sslots;
  bool fused_sq[DVM_MAX_NODES];   // x*x whose only consumer is a row sum: folded into that reduction
  bool fused_sc[DVM_MAX_NODES];   // per-row scalar muls/adds folded into a later multiply-add(-unary) instruction
  int8_t act_of[DVM_MAX_NODES];   // -1, or the fused activation (DVM_ACT_*) this node is the result of
  int16_t act_src[DVM_MAX_NODES]; // ... applied to this value
  bool act_part[DVM_MAX_NODES];   // an inner node of a fused activation chain: never materialises
  int16_t sel_src[DVM_MAX_NODES]; // -1, or: this Select chooses between two scalar multiples / offsets of value sel_src
  uint8_t sel_ar[DVM_MAX_NODES];  // ... DVM_A_MUL or DVM_A_ADD
  float sel_imm[DVM_MAX_NODES][2];
  int16_t n_cons[DVM_MAX_NODES];  // number of consuming nodes / outputs of a value
  int16_t one_cons[DVM_MAX_NODES];// the consuming node when there is exactly one (and it is a node)
  int lda_pos;                    // body position of the LDA just emitted by ensure_acc, or -1
  int8_t in_operand[DVM_MAX_NODES];
  bool stored[DVM_MAX_TENSORS];
  int8_t out_operand[DVM_MAX_TENSORS];
  const float* scalars;
  int n_scalars;
  bool fail;
  bool phased;                    // rows longer than a tile: the program runs in phases over column blocks (DVM_OP_PHASE)
  int n_phases;
};

static inline int root(const Enc& e, int v) {
  while (e.alias[v] >= 0) v = e.alias[v];
  return v;
}

static inline void emit(Enc& e, uint32_t w) { e.body[e.n_body++] = w; }

static inline uint32_t f2u(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  return u;
}

static int alloc_tmp(Enc& e) {  // a temporary local register (numbered after the input registers)
  for (int k = 0; k < DVM_MAX_LREGS - e.n_in_regs; ++k)
    if (e.tmp_val[k] < 0) {
      if (k + 1 > e.n_tmp_regs) e.n_tmp_regs = k + 1;
      return e.n_in_regs + k;
    }
  e.fail = true;
  return -1;
}

static int alloc_sreg(Enc& e) {
  for (int k = 0; k < DVM_MAX_SREGS; ++k)
    if (e.sreg_val[k] < 0) return k;
  e.fail = true;
  return -1;
}

static void release(Enc& e, int v) {  // free the registers of a dead value
  if (e.uses[v] > 0) return;
  if (e.cls[v] == CLS_TILE) {
    if (e.lreg_of[v] >= e.n_in_regs) {  // input registers stay bound to their input for the whole tile
      e.tmp_val[e.lreg_of[v] - e.n_in_regs] = -1;
      e.lreg_of[v] = -1;
    }
  } else if (e.sreg_of[v] >= 0 && !e.phased) {  // (a phased program's scalars outlive the tile: never recycled)
    e.sreg_val[e.sreg_of[v]] = -1;
    e.sreg_of[v] = -1;
  }
}

static void spill_acc_if_live(Enc& e) {
  int a = e.acc;
  if (a >= 0 && e.uses[a] > 0 && e.lreg_of[a] < 0) {
    int k = alloc_tmp(e);
    if (k < 0) return;
    emit(e, DVM_INSN(DVM_OP_STA, 1, k, 0));
    e.lreg_of[a] = (int8_t)k;
    e.ldt_of[a] = DVM_DT_F32;
    e.tmp_val[k - e.n_in_regs] = (int16_t)a;
  }
}

static void ensure_acc(Enc& e, int v) {
  if (e.acc == v) return;
  spill_acc_if_live(e);
  if (e.fail) return;
  if (e.lreg_of[v] >= 0) {
    e.lda_pos = e.n_body;
    emit(e, DVM_INSN(DVM_OP_LDA, 1, e.lreg_of[v], e.ldt_of[v]));
    e.acc = (int16_t)v;
  } else {
    e.fail = true;  // value was dropped: cannot happen with correct use counts
  }
}

static int ensure_sreg(Enc& e, int v) {
  if (e.sreg_of[v] >= 0) return e.sreg_of[v];
  if (e.sslot_of[v] >= 0) {
    int k = alloc_sreg(e);
    if (k < 0) return -1;
    emit(e, DVM_INSN(DVM_OP_LSS, 1, k, e.sslot_of[v]));
    e.sreg_of[v] = (int8_t)k;
    e.sreg_val[k] = (int16_t)v;
    return k;
  }
  e.fail = true;
  return -1;
}

static void store_outputs_of(Enc& e, int v) {  // value v is live in the accumulator (tile) or a scalar register
  for (int o = 0; o < e.p->n_outputs; ++o) {
    if (e.stored[o] || root(e, e.p->outputs[o].value) != v) continue;
    if (e.cls[v] == CLS_TILE) {
      ensure_acc(e, v);
      if (e.fail) return;
      emit(e, DVM_INSN(DVM_OP_STG, 1, 0, e.out_operand[o]));
    } else {
      int s = ensure_sreg(e, v);
      if (s < 0) return;
      emit(e, DVM_INSN(DVM_OP_STS, 1, s, e.out_operand[o]));
    }
    e.stored[o] = true;
    e.uses[v]--;
  }
}

static const uint8_t kBinMap[6] = {DVM_A_ADD, DVM_A_SUB, DVM_A_MUL, DVM_A_DIV, DVM_A_MIN, DVM_A_MAX};
static inline uint8_t reversed(uint8_t a) {
  if (a == DVM_A_SUB) return DVM_A_RSUB;
  if (a == DVM_A_DIV) return DVM_A_RDIV;
  return a;
}
static const uint8_t kUnMap[13] = {DVM_U_EXP, DVM_U_SQRT, DVM_U_RSQRT, DVM_U_ABS, DVM_U_LOG, DVM_U_ERF,
                                   DVM_U_SIGMOID, DVM_U_NEG, DVM_U_RECIP, DVM_U_FLOOR, DVM_U_ROUND, DVM_U_TANH,
                                   DVM_U_ISFINITE};

// Generates the load section (every global load of a tile, issued asynchronously into local
// registers before the tile is computed) and the compute section (accumulator code).
static bool gen_body(Enc& e) {
  const dvm_program* p = e.p;
  e.n_body = e.n_loads = 0;
  e.lda_pos = -1;
  e.fail = false;
  e.acc = -1;
  e.n_in_regs = e.n_tmp_regs = e.n_sslots = 0;
  for (int k = 0; k < DVM_MAX_LREGS; ++k) e.tmp_val[k] = -1;
  for (int k = 0; k < DVM_MAX_SREGS; ++k) e.sreg_val[k] = -1;
  for (int o = 0; o < p->n_outputs; ++o) e.stored[o] = false;
  for (int i = 0; i < p->n_nodes; ++i) {
    e.uses[i] = 0; e.lreg_of[i] = -1; e.sreg_of[i] = -1; e.sslot_of[i] = -1; e.ldt_of[i] = DVM_DT_F32;
    e.fused_sq[i] = false;
  }
  for (int i = 0; i < p->n_nodes; ++i) {
    const Node& n = p->nodes[i];
    if (n.kind == NK_INPUT || e.alias[i] >= 0) continue;
    e.uses[root(e, n.x)]++;
    if (n.kind == NK_BINARY || n.kind == NK_COMPARE || n.kind == NK_SELECT) e.uses[root(e, n.y)]++;
    if (n.kind == NK_SELECT) e.uses[root(e, n.param)]++;
  }
  for (int o = 0; o < p->n_outputs; ++o) e.uses[root(e, p->outputs[o].value)]++;
  // reduce_sum(x * x) with no other consumer of the square becomes one sum-of-squares reduction
  for (int i = 0; i < p->n_nodes; ++i) {
    const Node& n = p->nodes[i];
    if (n.kind != NK_REDUCE || n.op != DVM_SUM || e.alias[i] >= 0) continue;
    const int m = root(e, n.x);
    const Node& mn = p->nodes[m];
    if (mn.kind == NK_BINARY && mn.op == DVM_MUL && root(e, mn.x) == root(e, mn.y) && e.uses[m] == 1 &&
        e.cls[m] == CLS_TILE) {
      e.fused_sq[m] = true;
      e.uses[root(e, mn.x)] -= 1;  // the square consumed x twice, the fused reduction consumes it once
      e.uses[m] = 0;
    }
  }

  // Self-gating activations (pattern-based fusion, Sec. 5.1): the chains  0.5 * (t * (1 + erf(t / sqrt 2)))  and
  // t * sigmoid(t)  of single-consumer tile values become ONE instruction on t: no temporary has to keep t alive.
  for (int i = 0; i < p->n_nodes; ++i) { e.act_of[i] = -1; e.act_src[i] = -1; e.act_part[i] = false; }
  {
    auto is_imm = [&](const Node& n, int op, float v) {
      return n.kind == NK_SCALAR && n.op == op && n.param < 0 && fabsf(n.imm - v) <= 1e-6f * fabsf(v);
    };
    auto inner_ok = [&](int v) { return e.uses[v] == 1 && e.cls[v] == CLS_TILE && e.alias[v] < 0; };
    for (int i = 0; i < p->n_nodes; ++i) {
      const Node& n = p->nodes[i];
      if (e.alias[i] >= 0 || e.cls[i] != CLS_TILE) continue;
      if (is_imm(n, DVM_MULS, 0.5f)) {                          // 0.5 * m
        const int m = root(e, n.x);
        const Node& mn = p->nodes[m];
        if (mn.kind != NK_BINARY || mn.op != DVM_MUL || !inner_ok(m)) continue;
        for (int side = 0; side < 2; ++side) {                    // m = t * u3 or u3 * t
          const int t = root(e, side ? mn.y : mn.x), u3 = root(e, side ? mn.x : mn.y);
          if (t == u3 || e.cls[t] != CLS_TILE || !inner_ok(u3) || !is_imm(p->nodes[u3], DVM_ADDS, 1.0f)) continue;
          const int u2 = root(e, p->nodes[u3].x);
          if (!inner_ok(u2) || p->nodes[u2].kind != NK_UNARY || p->nodes[u2].op != DVM_ERF) continue;
          const int u1 = root(e, p->nodes[u2].x);
          if (!inner_ok(u1) || !is_imm(p->nodes[u1], DVM_MULS, 0.70710678f) || root(e, p->nodes[u1].x) != t) continue;
          e.act_of[i] = DVM_ACT_GELU; e.act_src[i] = (int16_t)t;
          e.act_part[m] = e.act_part[u3] = e.act_part[u2] = e.act_part[u1] = true;
          e.uses[m] = e.uses[u3] = e.uses[u2] = e.uses[u1] = 0;
          e.uses[t] -= 1;                                         // t fed u1 and m: the fused instruction reads it once
          break;
        }
      } else if (n.kind == NK_BINARY && n.op == DVM_MUL) {        // t * sigmoid(t)
        for (int side = 0; side < 2; ++side) {
          const int t = root(e, side ? n.y : n.x), s = root(e, side ? n.x : n.y);
          if (t == s || e.cls[t] != CLS_TILE || !inner_ok(s) || e.act_part[s] || p->nodes[s].kind != NK_UNARY ||
              p->nodes[s].op != DVM_SIGMOID || root(e, p->nodes[s].x) != t)
            continue;
          e.act_of[i] = DVM_ACT_SILU; e.act_src[i] = (int16_t)t;
          e.act_part[s] = true;
          e.uses[s] = 0;
          e.uses[t] -= 1;
          break;
        }
      }
    }
  }

  // Select(c, x * a, x * b) = x * Select(c, a, b), and the same with + : the two candidates never materialise
  for (int i = 0; i < p->n_nodes; ++i) e.sel_src[i] = -1;
  for (int i = 0; i < p->n_nodes; ++i) {
    const Node& n = p->nodes[i];
    if (n.kind != NK_SELECT || e.alias[i] >= 0 || e.cls[i] != CLS_TILE) continue;
    const int c = root(e, n.x), u = root(e, n.y), v = root(e, n.param);
    const Node& un = p->nodes[u];
    const Node& vn = p->nodes[v];
    if (u == v || un.kind != NK_SCALAR || vn.kind != NK_SCALAR || un.op != vn.op || e.uses[u] != 1 || e.uses[v] != 1 ||
        e.act_part[u] || e.act_part[v] || e.alias[u] >= 0 || e.alias[v] >= 0 || e.cls[u] != CLS_TILE || e.cls[v] != CLS_TILE)
      continue;
    const int x = root(e, un.x);
    if (x != root(e, vn.x) || x == c || e.cls[x] != CLS_TILE || e.cls[c] != CLS_TILE || p->nodes[x].kind != NK_INPUT) continue;
    e.sel_src[i] = (int16_t)x;
    e.sel_ar[i] = un.op == DVM_ADDS ? DVM_A_ADD : DVM_A_MUL;
    e.sel_imm[i][0] = un.param >= 0 ? e.scalars[un.param] : un.imm;
    e.sel_imm[i][1] = vn.param >= 0 ? e.scalars[vn.param] : vn.imm;
    e.act_part[u] = e.act_part[v] = true;  // (skipped like the inner nodes of a fused activation)
    e.uses[u] = e.uses[v] = 0;
    e.uses[x] -= 1;                        // x fed both candidates: the fused form reads it once
  }

  // consumers of every value (for the scalar multiply-add fusion below)
  for (int i = 0; i < p->n_nodes; ++i) { e.n_cons[i] = 0; e.one_cons[i] = -1; e.fused_sc[i] = false; }
  for (int i = 0; i < p->n_nodes; ++i) {
    const Node& n = p->nodes[i];
    if (n.kind == NK_INPUT || e.alias[i] >= 0 || e.fused_sq[i] || e.act_part[i]) continue;
    int x = root(e, n.x);
    if (e.act_of[i] >= 0) { e.n_cons[e.act_src[i]]++; e.one_cons[e.act_src[i]] = (int16_t)i; continue; }
    if (n.kind == NK_REDUCE && e.fused_sq[x]) x = root(e, p->nodes[x].x);
    e.n_cons[x]++; e.one_cons[x] = (int16_t)i;
    if (n.kind == NK_BINARY || n.kind == NK_COMPARE || n.kind == NK_SELECT) { int y = root(e, n.y); e.n_cons[y]++; e.one_cons[y] = (int16_t)i; }
    if (n.kind == NK_SELECT) { int z = root(e, n.param); e.n_cons[z]++; e.one_cons[z] = (int16_t)i; }
  }
  for (int o = 0; o < p->n_outputs; ++o) { int v = root(e, p->outputs[o].value); e.n_cons[v] += 2; }

  // ---- load section: one instruction per used input ----
  for (int ii = 0; ii < p->n_inputs; ++ii) {
    const int v = p->inputs[ii];
    if (e.uses[v] == 0) continue;
    const int od = e.in_operand[v];
    if (e.cls[v] == CLS_TILE) {
      if (e.n_in_regs >= DVM_MAX_LREGS - 1) return false;
      const int k = e.n_in_regs++;
      e.loads[e.n_loads++] = DVM_INSN(DVM_OP_LDG, 1, k, od);
      e.lreg_of[v] = (int8_t)k;
      e.ldt_of[v] = (int8_t)(e.opd[od].cs != 1 ? DVM_DT_F32 : e.opd[od].dtype);  // gathered elements are widened on the way in
    } else {
      if (e.n_sslots >= DVM_MAX_SSLOTS) return false;
      const int k = e.n_sslots++;
      e.loads[e.n_loads++] = DVM_INSN(DVM_OP_LDS, 1, k, od);
      e.sslot_of[v] = (int8_t)k;
    }
  }

  // ---- compute section ----
  for (int i = 0; i < p->n_nodes && !e.fail; ++i) {
    const Node& n = p->nodes[i];
    if (n.kind == NK_INPUT || e.alias[i] >= 0 || e.fused_sq[i] || e.act_part[i]) continue;
    int x = root(e, n.x);
    if (e.act_of[i] >= 0) {  // a fused activation of the value act_src: one instruction on the accumulator
      const int t = e.act_src[i];
      ensure_acc(e, t);
      if (e.fail) break;
      e.uses[t]--;
      spill_acc_if_live(e);
      if (e.fail) break;
      emit(e, DVM_INSN(DVM_OP_ACT + e.act_of[i], 1, 0, 0));
      e.acc = (int16_t)i;
      release(e, t);
      store_outputs_of(e, i);
      if (e.acc == i && e.uses[i] == 0) e.acc = -1;
      continue;
    }
    if (e.cls[i] == CLS_SCAL && (n.kind == NK_COMPARE || n.kind == NK_SELECT)) { e.fail = true; break; }
    if (e.cls[i] == CLS_SCAL && n.kind != NK_REDUCE) {
      // ---- per-row scalar arithmetic ----
      if (e.fused_sc[i]) continue;  // folded into the multiply-add instruction of a later node
      // s * m + a followed by a unary (the rstd of a norm, a mean) is ONE instruction: walk the chain of
      // single-consumer muls -> adds -> unary nodes that starts here
      if (n.kind == NK_SCALAR) {
        auto imm_of = [&](const Node& c) { return c.param >= 0 ? e.scalars[c.param] : c.imm; };
        int chain[3] = {i, -1, -1};
        int len = 1, un = 0xff;
        bool have_add = n.op == DVM_ADDS;
        float m = have_add ? 1.0f : imm_of(n), a = have_add ? imm_of(n) : 0.0f;
        int cur = i;
        while (len < 3) {
          const int nx = e.n_cons[cur] == 1 ? e.one_cons[cur] : -1;
          if (nx < 0 || e.cls[nx] != CLS_SCAL || root(e, p->nodes[nx].x) != cur) break;
          const Node& nn = p->nodes[nx];
          if (nn.kind == NK_SCALAR && nn.op == DVM_ADDS && !have_add) {
            a = imm_of(nn);
            have_add = true;
            chain[len++] = nx;
            cur = nx;
          } else if (nn.kind == NK_UNARY) {
            un = kUnMap[nn.op];
            chain[len++] = nx;
            break;
          } else {
            break;
          }
        }
        if (len >= 2) {
          const int last = chain[len - 1];
          int sx = ensure_sreg(e, x);
          if (e.fail) break;
          e.uses[x]--;
          release(e, x);
          int d = alloc_sreg(e);
          if (d < 0) break;
          emit(e, DVM_INSN(DVM_OP_SOP, 4, d, DVM_SK_FMAU));
          emit(e, (uint32_t)un | ((uint32_t)sx << 8));
          emit(e, f2u(m));
          emit(e, f2u(a));
          for (int q = 0; q < len; ++q) e.fused_sc[chain[q]] = true;   // later chain nodes are skipped
          for (int q = 0; q + 1 < len; ++q) e.uses[chain[q]] = 0;       // intermediates never materialise
          e.sreg_of[last] = (int8_t)d;
          e.sreg_val[d] = (int16_t)last;
          store_outputs_of(e, last);
          release(e, last);
          continue;
        }
      }
      int sx = ensure_sreg(e, x);
      int sy = -1;
      int y = -1;
      if (n.kind == NK_BINARY) { y = root(e, n.y); sy = ensure_sreg(e, y); }
      if (e.fail) break;
      e.uses[x]--;
      if (y >= 0) e.uses[y]--;
      release(e, x);
      if (y >= 0 && y != x) release(e, y);
      int d = alloc_sreg(e);
      if (d < 0) break;
      if (n.kind == NK_BINARY) {
        emit(e, DVM_INSN(DVM_OP_SOP, 2, d, DVM_SK_BIN));
        emit(e, (uint32_t)kBinMap[n.op] | ((uint32_t)sx << 8) | ((uint32_t)sy << 16));
      } else if (n.kind == NK_SCALAR) {
        float s = n.param >= 0 ? e.scalars[n.param] : n.imm;
        emit(e, DVM_INSN(DVM_OP_SOP, 3, d, DVM_SK_BINI));
        emit(e, (uint32_t)(n.op == DVM_ADDS ? DVM_A_ADD : DVM_A_MUL) | ((uint32_t)sx << 8));
        emit(e, f2u(s));
      } else {  // unary or rounding cast
        uint32_t u = n.kind == NK_CAST ? (uint32_t)(n.dtype == DVM_I32 ? DVM_U_TRUNC_I32 : n.dtype == DVM_U8 ? DVM_U_TRUNC_U8 : DVM_U_RND_BF16)
                                       : (uint32_t)kUnMap[n.op];
        emit(e, DVM_INSN(DVM_OP_SOP, 2, d, DVM_SK_UN));
        emit(e, u | ((uint32_t)sx << 8));
      }
      e.sreg_of[i] = (int8_t)d;
      e.sreg_val[d] = (int16_t)i;
      store_outputs_of(e, i);
      release(e, i);
      continue;
    }
    if (n.kind == NK_REDUCE) {
      const bool sq = e.fused_sq[x];
      if (sq) x = root(e, p->nodes[x].x);
      ensure_acc(e, x);
      if (e.fail) break;
      e.uses[x]--;
      int d = alloc_sreg(e);
      if (d < 0) break;
      emit(e, DVM_INSN(DVM_OP_RED + (sq ? DVM_R_SUMSQ : n.op == DVM_SUM ? DVM_R_SUM : n.op == DVM_RMAX ? DVM_R_MAX : DVM_R_MIN),
                       1, d, 0));
      e.sreg_of[i] = (int8_t)d;
      e.sreg_val[d] = (int16_t)i;
      release(e, x);
      store_outputs_of(e, i);
      release(e, i);
      continue;
    }
    // ---- tile-class result in the accumulator ----
    if (n.kind == NK_COMPARE) {
      // ACC = ACC cmp L[b]; with the right operand in the accumulator the relation is mirrored
      static const uint8_t kMirror[8] = {DVM_C_LT, DVM_C_LE, DVM_C_GT, DVM_C_GE, DVM_C_EQ, DVM_C_NE, DVM_C_RPOW, DVM_C_POW};
      const int y = root(e, n.y);
      if (e.cls[i] != CLS_TILE || e.cls[x] != CLS_TILE || e.cls[y] != CLS_TILE) { e.fail = true; break; }
      int a = x, b = y;
      uint8_t cop = n.op;
      if (e.acc == y && e.acc != x) { a = y; b = x; cop = kMirror[cop]; }
      ensure_acc(e, a);
      if (e.fail) break;
      const int bk = b == a ? 0xff : e.lreg_of[b];
      if (bk < 0) { e.fail = true; break; }
      e.uses[a]--;
      e.uses[b]--;
      spill_acc_if_live(e);
      if (e.fail) break;
      emit(e, DVM_INSN(DVM_OP_CMP + cop, 1, bk, b == a ? DVM_DT_F32 : e.ldt_of[b]));
      e.acc = (int16_t)i;
      release(e, a);
      if (b != a) release(e, b);
    } else if (n.kind == NK_SELECT && e.sel_src[i] >= 0) {
      // the scalar is selected in the accumulator, then applied to x (an input: it has a local register)
      const int xs = e.sel_src[i];
      if (e.lreg_of[xs] < 0) { e.fail = true; break; }
      ensure_acc(e, x);
      if (e.fail) break;
      e.uses[x]--;
      spill_acc_if_live(e);
      if (e.fail) break;
      emit(e, DVM_INSN(DVM_OP_SEL + 3, 3, 0, 0));
      emit(e, f2u(e.sel_imm[i][0]));
      emit(e, f2u(e.sel_imm[i][1]));
      emit(e, DVM_INSN(DVM_OP_BIN + e.sel_ar[i], 1, e.lreg_of[xs], e.ldt_of[xs]));
      e.uses[xs]--;
      e.acc = (int16_t)i;
      release(e, x);
      release(e, xs);
    } else if (n.kind == NK_SELECT) {
      // one of {condition, then-value, else-value} stays in (or moves to) the accumulator, the other two are
      // read from local registers
      const int xv = root(e, n.y), yv = root(e, n.param);
      if (e.cls[i] != CLS_TILE || e.cls[x] != CLS_TILE || e.cls[xv] != CLS_TILE || e.cls[yv] != CLS_TILE) { e.fail = true; break; }
      int form = 0, in_acc = x, p1 = xv, p2 = yv;             // 0x58: condition in ACC, L[then], L[else]
      if (e.acc == yv && yv != x) { form = 1; in_acc = yv; p1 = x; p2 = xv; }        // 0x59: L[cond], L[then], else in ACC
      else if (e.acc == xv && xv != x) { form = 2; in_acc = xv; p1 = x; p2 = yv; }   // 0x5a: L[cond], then in ACC, L[else]
      ensure_acc(e, in_acc);
      if (e.fail) break;
      const int rd[2] = {p1, p2};
      for (int q = 0; q < 2 && !e.fail; ++q) {
        const int v = rd[q];
        if (e.lreg_of[v] >= 0) continue;
        if (e.acc != v) { e.fail = true; break; }
        const int k = alloc_tmp(e);  // also the accumulator's value: keep a copy in a local register
        if (k < 0) break;
        emit(e, DVM_INSN(DVM_OP_STA, 1, k, 0));
        e.lreg_of[v] = (int8_t)k;
        e.ldt_of[v] = DVM_DT_F32;
        e.tmp_val[k - e.n_in_regs] = (int16_t)v;
      }
      if (e.fail) break;
      e.uses[x]--;
      e.uses[xv]--;
      e.uses[yv]--;
      spill_acc_if_live(e);
      if (e.fail) break;
      emit(e, DVM_INSN(DVM_OP_SEL + form, 1, e.lreg_of[p1],
                       (uint32_t)e.lreg_of[p2] | ((uint32_t)e.ldt_of[p1] << 6) | ((uint32_t)e.ldt_of[p2] << 7)));
      e.acc = (int16_t)i;
      release(e, x);
      if (xv != x) release(e, xv);
      if (yv != x && yv != xv) release(e, yv);
    } else if (n.kind == NK_BINARY) {
      int y = root(e, n.y);
      uint8_t ar = kBinMap[n.op];
      int a = x, b = y;  // a: accumulator operand, b: the other
      bool swap = false;
      if (e.cls[x] == CLS_SCAL) swap = true;                                   // scalar (op) tile
      else if (e.cls[y] == CLS_TILE && e.acc == y && e.acc != x) swap = true;   // right operand already in the accumulator
      if (swap) { a = y; b = x; ar = reversed(ar); }
      ensure_acc(e, a);
      if (e.fail) break;
      int bk = -1;
      if (e.cls[b] == CLS_TILE) {
        if (b == a) bk = 0xff;
        else if (e.lreg_of[b] >= 0) bk = e.lreg_of[b];
        else e.fail = true;
      } else {
        bk = ensure_sreg(e, b);
      }
      if (e.fail || bk < 0) { e.fail = true; break; }
      e.uses[a]--;
      e.uses[b]--;
      spill_acc_if_live(e);
      if (e.fail) break;
      if (e.cls[b] == CLS_TILE) {
        if (b != a && e.lda_pos == e.n_body - 1) {
          // the accumulator was loaded just for this operation: one fused instruction ACC = L[x] op L[y]
          const uint32_t lda = e.body[e.lda_pos];
          e.body[e.lda_pos] = DVM_INSN(DVM_OP_LD2 + ar, 1, DVM_INSN_A(lda),
                                       (uint32_t)bk | (DVM_INSN_B(lda) << 6) | ((uint32_t)e.ldt_of[b] << 7));
          e.lda_pos = -1;
        } else {
          emit(e, DVM_INSN(DVM_OP_BIN + ar, 1, bk, b == a ? DVM_DT_F32 : e.ldt_of[b]));
        }
      } else {
        emit(e, DVM_INSN(DVM_OP_BINS + ar, 1, bk, 0));
      }
      e.acc = (int16_t)i;
      release(e, a);
      if (b != a) release(e, b);
    } else {
      ensure_acc(e, x);
      if (e.fail) break;
      e.uses[x]--;
      spill_acc_if_live(e);
      if (e.fail) break;
      if (n.kind == NK_UNARY) {
        emit(e, DVM_INSN(DVM_OP_UN + kUnMap[n.op], 1, 0, 0));
      } else if (n.kind == NK_SCALAR) {
        float s = n.param >= 0 ? e.scalars[n.param] : n.imm;
        emit(e, DVM_INSN(DVM_OP_BINI + (n.op == DVM_ADDS ? DVM_A_ADD : DVM_A_MUL), 2, 0, 0));
        emit(e, f2u(s));
      } else {  // NK_CAST to bf16 or to an integer type (casts to f32 are aliases)
        emit(e, DVM_INSN(DVM_OP_UN + (n.dtype == DVM_I32 ? DVM_U_TRUNC_I32 : n.dtype == DVM_U8 ? DVM_U_TRUNC_U8 : DVM_U_RND_BF16), 1, 0, 0));
      }
      e.acc = (int16_t)i;
      release(e, x);
    }
    store_outputs_of(e, i);
    if (e.acc == i && e.uses[i] == 0) e.acc = -1;
  }
  if (e.fail) return false;
  // outputs that are inputs (or aliases of inputs)
  for (int o = 0; o < p->n_outputs && !e.fail; ++o)
    if (!e.stored[o]) store_outputs_of(e, root(e, p->outputs[o].value));
  return !e.fail;
}

// Rows longer than a tile (DVM_OP_PHASE).  The compute section was generated for one tile; every tile of a row
// walks it again, so what a tile computes must depend only on the tile's own loads and on per-row scalars that are
// complete.  This pass follows the code once, notes in which phase each value becomes available -- a tile value
// as early as its operands, a reduction one phase after the value it reduces -- tags the instructions that must
// run once (RED in the phase of its operand; scalar arithmetic and scalar stores in the last block of the phase
// that completes their operands; tile stores in the last phase), cuts every phase's walk off behind the last
// instruction it needs, and puts the phase count in front.
static bool tag_phases(Enc& e) {
  int lreg_av[DVM_MAX_LREGS], s_ready[DVM_MAX_SREGS];
  for (int k = 0; k < DVM_MAX_LREGS; ++k) lreg_av[k] = 0;
  for (int k = 0; k < DVM_MAX_SREGS; ++k) s_ready[k] = -1;  // -1: ready from the first tile on (a loaded per-row value)
  int acc_av = 0, P = 1;
  auto after = [](int ready) { return ready + 1; };  // first phase that may read a scalar completed in phase `ready`
  for (int pass = 0; pass < 2; ++pass) {
    acc_av = 0;
    for (int pc = 0; pc < e.n_body;) {
      uint32_t w0 = e.body[pc];
      const uint32_t op = DVM_INSN_OP(w0), a = DVM_INSN_A(w0), b = DVM_INSN_B(w0);
      const int len = (int)DVM_INSN_LEN(w0);
      int tag = 0;
      if (op == DVM_OP_LDA) acc_av = lreg_av[a];
      else if (op == DVM_OP_STA) lreg_av[a] = acc_av;
      else if (op == DVM_OP_LSS) s_ready[a] = -1;
      else if (op == DVM_OP_BCS) acc_av = after(s_ready[a]);
      else if (op >= DVM_OP_LD2 && op < DVM_OP_LD2 + DVM_A_NBIN) acc_av = std::max(lreg_av[a], lreg_av[b & 0x3f]);
      else if ((op >= DVM_OP_BIN && op < DVM_OP_BIN + DVM_A_NBIN) || (op >= DVM_OP_CMP && op < DVM_OP_CMP + DVM_C_NCMP)) {
        if (a != DVM_REG_ACC) acc_av = std::max(acc_av, lreg_av[a]);
      } else if (op >= DVM_OP_SEL && op < DVM_OP_SEL + 3) acc_av = std::max(acc_av, std::max(lreg_av[a], lreg_av[b & 0x3f]));
      else if (op >= DVM_OP_BINS && op < DVM_OP_BINS + DVM_A_NBIN) acc_av = std::max(acc_av, after(s_ready[a]));
      else if (op >= DVM_OP_RED && op < DVM_OP_RED + DVM_R_NRED) {
        tag = acc_av + 1;
        s_ready[a] = acc_av;
        P = std::max(P, acc_av + 1);
      } else if (op == DVM_OP_SOP) {
        const uint32_t w1 = e.body[pc + 1];
        int j = s_ready[(w1 >> 8) & 0xff];
        if (b == DVM_SK_BIN) j = std::max(j, s_ready[(w1 >> 16) & 0xff]);
        tag = j < 0 ? 0 : j + 1;  // from loaded values only: every tile may repeat it
        s_ready[a] = j;
      } else if (op == DVM_OP_STS) {
        tag = std::max(s_ready[a], 0) + 1;
      } else if (op == DVM_OP_STG) {
        P = std::max(P, acc_av + 1);
        tag = P;  // (final in the second pass)
      }
      if (pass == 1 && tag) e.body[pc] = DVM_INSN_SET_TAG(w0, tag);
      pc += len;
    }
    if (P > DVM_MAX_PHASES) return false;
  }
  // the walk of phase k ends behind the last instruction tagged for a phase <= k
  uint32_t out[sizeof(e.body) / sizeof(e.body[0])];
  int n = 0, cut[DVM_MAX_PHASES];
  for (int k = 0; k + 1 < P; ++k) cut[k] = 0;
  for (int pc = 0; pc < e.n_body; pc += (int)DVM_INSN_LEN(e.body[pc])) {
    const int t = (int)DVM_INSN_TAG(e.body[pc]);
    for (int k = 0; k + 1 < P; ++k)
      if (t && t - 1 <= k) cut[k] = pc + (int)DVM_INSN_LEN(e.body[pc]);
  }
  if (e.n_body + P + 1 > (int)(sizeof(e.body) / sizeof(e.body[0]))) return false;
  out[n++] = DVM_INSN(DVM_OP_PHASE, 1, 0xff, P);
  for (int pc = 0; pc < e.n_body;) {
    const int len = (int)DVM_INSN_LEN(e.body[pc]);
    for (int q = 0; q < len; ++q) out[n++] = e.body[pc + q];
    pc += len;
    for (int k = 0; k + 1 < P; ++k)
      if (cut[k] == pc) out[n++] = DVM_INSN(DVM_OP_PHASE, 1, k + 1, 0);
  }
  memcpy(e.body, out, (size_t)n * 4);
  e.n_body = n;
  e.n_phases = P;
  return true;
}

}  // namespace

int dvm_encode_matmul(const dvm_program* p, const dvm_shape* in_shapes, int n_in, const float* scalars,
                      int n_scalars, void* code, size_t code_capacity, size_t* code_size,
                      dvm_shape* out_shapes, int n_out);

// in_strides / out_strides (each may be NULL: dense row-major): element strides of the views (ViewLoad /
// ViewStore, Table 1), one entry per input / output.
// `combine_axis` (0: none; else the reduced axis, counted from the end): the program's reductions are results
// only -- they become plain tile values that every tile combines into the result with atomic operations
// (the stored view has stride 0 along the reduced axis: all its rows land on one address).
// `lowered`: the shapes are those of encode_views' axis permutation (rank of the dominant shape, not the
// inputs' declared ranks); every reduction then runs over the last dim.
// What steps 1 - 5 of the encoder hand to the shape tiling and to the assembly: the collapsed iteration space and
// the registers the generated code uses.
struct Lowered {
  int64_t C, R, outer[3];        // columns, rows and the (up to three) collapsed outer dims of the dominant shape
  bool flat, empty, has_reduce;
  int primary, combine_axis, W, nreg;
  int in_dtype[DVM_MAX_LREGS], in_opd[DVM_MAX_LREGS];  // element type and operand of every input register
};

// One candidate of the shape tiling, with the local-memory layout of its tile slot.
struct Geo {
  int V, log2G, W, units, scalar_unit;
  bool one_slot;  // costed for two CTAs per SM that hold ONE tile slot each (see DVM_F_ONE_SLOT)
  int64_t Ctile, CB, rowsR, lastRowCols, n_tiles, cost;
  uint32_t flags, inv_mask;
  uint32_t lreg_table[DVM_MAX_LREGS];
};

// Step 6 of the encoder: the shape tiling.  Leaves the cheapest geometry in `best`.
static int choose_geometry(const Enc& e, const Lowered& L, Geo& best) {
  const dvm_program* p = e.p;
  const int NN = p->n_nodes;
  const bool flat = L.flat, empty = L.empty, has_reduce = L.has_reduce;
  const int64_t C = L.C, R = L.R;
  const int64_t* outer = L.outer;
  const int W = L.W, primary = L.primary, combine_axis = L.combine_axis, nreg = L.nreg;
  const int* in_dtype = L.in_dtype;
  const int* in_opd = L.in_opd;
  // ---- 6. shape tiling (Sec. 4.2): elements per thread V, threads per row G, column tile, tile count.
  // Candidates are compared with the paper's cost  ceil(#tiles / N) * (tile + overhead)  in per-thread
  // element units; N is the number of CTAs resident at once, which the local-memory need decides.
  const int T = DVM_VM_THREADS;
  const int64_t beta = 12;  // per-tile decode overhead in element units (the paper's "+2")
  Geo tight;  // the best geometry among those that leave room for g_min_resident_ctas CTAs per SM
  best.cost = -1;
  tight.cost = -1;
  // Local-memory layout of ONE tile slot, in 256-byte units, for a candidate geometry; returns the CTAs per SM
  // it leaves room for (0: it does not fit at all).  An input register is an image of the tile's rows as they
  // lie in global memory (a dense operand: one contiguous range; otherwise one image per row, DVM_ROW_PITCH
  // apart; a row vector shared by every row: one row image, of the tile's column block); a temporary is
  // thread-private (V fp32 per thread); per-row scalar slots are thread-private.  A CTA holds two slots:
  // while it computes the tile in one, the next tile (of this or of another stacked program) loads into the
  // other.
  auto layout = [&](Geo& g) -> int {
    g.inv_mask = 0;
    g.units = 0;
    const int64_t Gthreads = 1ll << g.log2G;
    for (int k = 0; k < e.n_in_regs; ++k) {
      const Operand& od = e.opd[in_opd[k]];
      const int es = in_dtype[k] == DVM_DT_BF16 ? 2 : 4;
      const bool inv = !flat && od.ostride[0] == 0 && od.ostride[1] == 0 && od.ostride[2] == 0;
      const bool gather = od.col_stride == 1 && od.cs != 1;
      bool dense = od.col_stride == 1 && od.cs == 1 && od.ostride[0] == (flat ? g.Ctile : C) && g.CB == 1;
      if (!flat) {
        if (outer[1] > 1 && od.ostride[1] != od.ostride[0] * outer[0]) dense = false;
        if (outer[2] > 1 && od.ostride[2] != od.ostride[1] * outer[1]) dense = false;
      }
      // a gathered operand whose rows are adjacent in memory (a transposed matrix): with few threads per row the
      // tile's part of a column is a contiguous strip of 256 / G elements -- copied in bulk, one strip per column
      bool transposed = gather && !flat && !e.phased && od.ostride[0] == 1 && (od.cs * es) % 16 == 0 &&
                        Gthreads * g.V <= T && ((T / Gthreads) * es) % 16 == 0;
      for (int q = 1; q < 3 && transposed; ++q)
        if (outer[q] > 1 && ((od.ostride[q] * es) % 16 != 0 || outer[0] % (T / Gthreads) != 0)) transposed = false;
      const int mode = transposed ? DVM_LM_TRANSPOSED : gather ? DVM_LM_GATHER
                              : (inv ? (g.CB == 1 ? DVM_LM_BCAST : DVM_LM_BCAST_TILE) : (dense ? DVM_LM_BLOCK : DVM_LM_ROWS));
      if (inv && !gather) g.inv_mask |= 1u << k;  // one column block: the same for every tile, loaded once per slot
      const int64_t pitch = DVM_ROW_PITCH(Gthreads, g.V, es);
      // a gathered register holds fp32 values in the thread-private layout of a temporary
      const int64_t bytes = transposed ? g.Ctile * (int64_t)DVM_STRIP_PITCH(T / Gthreads, es)
                                       : gather ? (int64_t)g.V * 4 * T : (inv ? pitch : pitch * (T / Gthreads));
      g.lreg_table[k] = (uint32_t)g.units | ((uint32_t)mode << 16) | ((uint32_t)in_opd[k] << 24);
      g.units += (int)cdiv(bytes, DVM_LOCAL_UNIT);
    }
    for (int k = e.n_in_regs; k < nreg; ++k) {
      g.lreg_table[k] = (uint32_t)g.units | ((uint32_t)DVM_LM_PRIVATE << 16);
      g.units += g.V * 4 * T / DVM_LOCAL_UNIT;
    }
    g.scalar_unit = g.units;
    if (e.n_sslots > 0) g.units += 2 * 16 * T / DVM_LOCAL_UNIT;  // 8 fp32 slots per thread
    g.one_slot = false;
    if (g_stack_one_slot) {  // a stacked launch whose CTAs hold one tile slot: what has to fit twice is one slot
      if (g.units + 1 > DVM_MAX_LOCAL_UNITS / 2) return g.units + 1 > DVM_MAX_LOCAL_UNITS ? 0 : 1;
      const int one = 233472 / ((g.units + 1) * DVM_LOCAL_UNIT + 9600);
      return one > 2 ? 2 : one;
    }
    if (2 * g.units + 1 > DVM_MAX_LOCAL_UNITS) return 0;
    int ctas = 233472 / ((2 * g.units + 1) * DVM_LOCAL_UNIT + 9600);  // 228 KB per SM; per CTA: 1 KB reserved + 8.3 KB static
    if (ctas == 1 && g.V != 24 && g_min_resident_ctas < 2 && !e.phased && 233472 / ((g.units + 1) * DVM_LOCAL_UNIT + 9600) >= 2) {
      // Two slots fit once per SM, one slot fits twice: eight more warps per SM are worth more than the
      // prefetch inside a CTA (the other CTA computes while this one waits for its tile).  Only a launch of
      // the program on its own can honour this; the programs of a stacked launch share two slots.
      g.one_slot = true;
      return 2;
    }
    return ctas > 2 ? 2 : ctas;  // the interpreter is compiled for two resident CTAs per SM
  };
  // cores the tiles spread over when `ctas` CTAs are resident per SM (the core count is quoted at 3 CTAs per SM)
  auto cores = [&](int ctas) -> int64_t { return (int64_t)dvm_get_num_cores() * ctas / 3; };
  const int W0 = W;
  // 24 elements per thread (rows that fill three quarters of a 32-element tile) exist as the one-program
  // basic interpreter variant only: not for programs of stacked launches, not with Cmp / Select / views
  bool plain = g_min_resident_ctas == 0 && !combine_axis && !e.phased;
  for (int i = 0; i < NN; ++i) {
    const Node& n = p->nodes[i];
    if (n.kind == NK_COMPARE || n.kind == NK_SELECT || (n.kind == NK_UNARY && n.op == DVM_ISFINITE)) plain = false;
  }
  for (int o = 0; o < e.n_opd; ++o) {
    const Operand& od = e.opd[o];
    if (od.col_stride != 1) continue;
    bool dense = od.cs == 1 && (od.ostride[0] == C || outer[0] == 1);
    if (outer[1] > 1 && od.ostride[1] != od.ostride[0] * outer[0]) dense = false;
    if (outer[2] > 1 && od.ostride[2] != od.ostride[1] * outer[1]) dense = false;
    if (od.cs != 1 || (o >= e.n_opd - p->n_outputs && !dense && !flat)) plain = false;
  }
  static const int kVs[3] = {32, 24, 16};
  for (int vi = 0; vi < 3; ++vi) {
    Geo g;
    g.V = kVs[vi];
    if (g_elems_per_thread && g.V != g_elems_per_thread) continue;
    if (g.V == 24 && !plain && g_elems_per_thread != 24) continue;
    // a phased program walks a row P times: the fewest, largest column blocks keep the per-tile overhead and the
    // ragged last block small (8200 columns: 2 blocks of 4104 instead of 3 of 4096 / 4096 / 8)
    if (e.phased && g.V != 32 && !g_elems_per_thread) continue;
    g.W = W0;
    if (flat) {
      g.log2G = 8;
      g.CB = 1;
      g.Ctile = (int64_t)T * W0;  // the layout of a flat program does not depend on the chunk
      g.flags = DVM_F_FLAT | DVM_F_ALIGNED;
      const int ctas = layout(g);
      if (ctas < 1) continue;
      const int64_t N = cores(ctas);
      int64_t total = empty ? 0 : C;  // everything merged into one dim
      int64_t best_chunk = (int64_t)T * W0;
      g.cost = -1;
      for (int k = 1; k <= g.V / W0; ++k) {
        int64_t chunk = (int64_t)T * W0 * k;
        int64_t cost = cdiv(cdiv(total, chunk), N) * (W0 * k + beta);
        // a program of a stacked launch has no waves of its own: its cost is its total work, and a tile costs its
        // V slots whether the chunk fills them or not (half-filled chunks doubled sigmoid(x) * y: 117 -> instructions
        // per element in the C4 mix)
        if (g_min_resident_ctas == 2) cost = cdiv(total, chunk) * (g.V + beta);
        if (g.cost < 0 || cost <= g.cost) { g.cost = cost; best_chunk = chunk; }
      }
      g.Ctile = best_chunk;
      g.rowsR = cdiv(total, g.Ctile);
      g.lastRowCols = g.rowsR > 0 ? total - (g.rowsR - 1) * g.Ctile : g.Ctile;
      g.n_tiles = g.rowsR;
      layout(g);  // dense operands are recognised by the final chunk
      if (best.cost < 0 || g.cost < best.cost) best = g;
      if (ctas >= g_min_resident_ctas && (tight.cost < 0 || g.cost < tight.cost)) tight = g;
      continue;
    }
    // rows of the primary operand start on W-element boundaries (given an aligned base pointer)?
    bool aligned = primary >= 0;
    if (primary >= 0)
      for (int q = 0; q < 3; ++q)
        if (outer[q] > 1 && (e.opd[primary].ostride[q] % W0) != 0) aligned = false;
    const int w = W0;
    // a misaligned row segment starts up to w - 1 slots into its first chunk: keep that much spare capacity
    const int64_t pad = aligned ? 0 : w - 1;
    g.flags = (aligned ? DVM_F_ALIGNED : 0) | ((outer[1] > 1 || outer[2] > 1) ? DVM_F_OUTER_DIMS : 0);
    g.rowsR = R;
    g.lastRowCols = C;
    for (int lg = 8; lg >= 0; --lg) {  // ties go to more threads per row: wider coalesced accesses
      // combined results: the rows a warp holds (32 / G of them) are combined by shuffles before the atomics
      if (combine_axis && lg > 5) continue;
      int64_t G = 1 << lg, cap = G * g.V;
      // ... but not so few threads per row that a row copy shrinks below 512 bytes while the rows are wider
      // (measured on column sums: 256-byte copies 1560 GB/s, 512 bytes 1640, 1 KB and more lose to the atomics)
      if (combine_axis && cap * 4 < 512 && C * 4 >= 512) continue;
      if (e.phased && lg != 8) continue;  // one row per tile: the whole CTA on a column block
      int64_t ct;
      if (has_reduce && !e.phased) {
        // a whole row per thread group; at the widest group a row may use the full capacity: its last
        // columns then wrap around into the head slots of a misaligned row
        if (cap < C + pad && !(lg == 8 && cap >= C)) continue;
        ct = C;
      } else {
        ct = ((cap - pad) / w) * w;
        if (ct <= 0) continue;
        if (ct > C) ct = C;
        if (e.phased) ct = cdiv(cdiv(C, cdiv(C, ct)), w) * w;  // column blocks of even length
      }
      g.log2G = lg;
      g.Ctile = ct;
      g.CB = cdiv(C, ct);
      g.n_tiles = cdiv(R, T / G) * g.CB * e.n_phases;
      // the local-memory need of this geometry decides how many CTAs are resident at once
      const int ctas = layout(g);
      if (ctas < 1) continue;
      // elements one thread processes per tile: the interpreter walks all V slots of a tile register, used or
      // not (a row that fills three quarters of 32 slots costs what a full one costs: hence the 24-slot variant)
      int64_t u = g.V;
      g.cost = cdiv(g.n_tiles, cores(ctas)) * (u + beta + (combine_axis ? 2 * g.V * G / 32 : 0));  // + the atomics a thread issues
      if (g_min_resident_ctas == 2) {
        // A program of a stacked launch shares the machine with the launch's other programs: there are no
        // waves of its own to fill, what counts is its total work -- tiles x (elements per thread + overhead).
        // (A term for the row copies a tile issues was measured and did not pay: narrower tiles that waste
        // fewer slots win even at 64 copies of 256 bytes per tile.)
        g.cost = g.n_tiles * (u + beta);
      }
      // Gathered / scattered operands whose ROWS are adjacent in memory (a transposed matrix): a warp's 32
      // lanes cover min(32, G) columns x 32 / min(32, G) consecutive rows, and only the rows share 32-byte
      // sectors -- few threads per row keep the traffic near the algorithmic bytes, many multiply it.
      {
        int64_t num = 0, den = 0;
        for (int o = 0; o < e.n_opd; ++o) {
          const Operand& od = e.opd[o];
          if (od.col_stride != 1) continue;
          const int64_t es = (int64_t)1 << DVM_DT_LG_ES(od.dtype);
          int64_t amp = 4;  // in quarters: 4 = no amplification
          if (od.cs > 1 && od.ostride[0] == 1) {
            const int64_t nT = G < 32 ? G : 32, nR = 32 / nT;
            amp = 4 * nT * cdiv(nR * es, 32) * 32 / (32 * es);
            if (amp < 4) amp = 4;
          }
          num += amp * es;
          den += 4 * es;
        }
        if (den > 0) g.cost = g.cost * num / den;
      }
      if (empty) g.n_tiles = 0;
      if (best.cost < 0 || g.cost < best.cost) best = g;
      if (ctas >= g_min_resident_ctas && (tight.cost < 0 || g.cost < tight.cost)) tight = g;
    }
  }
  if (tight.cost >= 0) best = tight;  // otherwise no geometry leaves that room: the unconstrained best stands
  if (best.cost < 0) return DVM_ERR_UNSUPPORTED;  // row longer than the register budget, or too much local memory
  return DVM_OK;
}

// Step 7 of the encoder: flags, header, tables and code of the chosen geometry into the caller's buffer.
static int assemble_program(Enc& e, const Lowered& L, const Geo& best, int n_in, void* code, size_t code_capacity,
                            size_t* code_size) {
  const dvm_program* p = e.p;
  const int NN = p->n_nodes;
  const bool flat = L.flat;
  const int primary = L.primary, nreg = L.nreg;
  int W = L.W;
  int64_t C = L.C;
  int64_t outer[3] = {L.outer[0], L.outer[1], L.outer[2]};
  const int log2G = best.log2G;
  W = best.W;
  const int64_t Ctile = best.Ctile, CB = best.CB, rowsR = best.rowsR, lastRowCols = best.lastRowCols, n_tiles = best.n_tiles;
  uint32_t flags = best.flags;
  const int units = best.units, scalar_unit = best.scalar_unit;
  const uint32_t* lreg_table = best.lreg_table;
  if (flat) {
    C = Ctile;
    for (int o = 0; o < e.n_opd; ++o) {
      e.opd[o].ostride[0] = e.opd[o].col_stride ? Ctile * e.opd[o].cs : 0;
      e.opd[o].ostride[1] = e.opd[o].ostride[2] = 0;
    }
    outer[0] = rowsR; outer[1] = outer[2] = 1;
  }
  if (n_tiles > 0xffffffffll || rowsR > 0xffffffffll) return DVM_ERR_TOO_LARGE;

  // dense operands: the rows of a tile are one contiguous range (flat offset = row * C + col)
  bool dense_of[DVM_MAX_OPERANDS];
  for (int o = 0; o < e.n_opd; ++o) {
    const Operand& od = e.opd[o];
    bool dense = od.col_stride == 1 && od.cs == 1 && (od.ostride[0] == C || outer[0] == 1);  // (a single row has no stride)
    if (outer[1] > 1 && od.ostride[1] != od.ostride[0] * outer[0]) dense = false;
    if (outer[2] > 1 && od.ostride[2] != od.ostride[1] * outer[1]) dense = false;
    dense_of[o] = dense;
  }
  if (primary >= 0 && dense_of[primary]) flags |= DVM_F_PRIMARY_DENSE;
  if (primary < 0) flags |= DVM_F_ALIGNED;  // no tile-class memory operand: nothing to align to
  if (best.one_slot) flags |= DVM_F_ONE_SLOT;
  if (e.n_sslots > 0) flags |= DVM_F_LOADS_BY_ROW;
  for (int i = 0; i < NN; ++i)
    if (p->nodes[i].kind == NK_COMPARE || p->nodes[i].kind == NK_SELECT) flags |= DVM_F_EXT_ISA;
  for (int i = 0; i < NN; ++i)
    if (p->nodes[i].kind == NK_UNARY && p->nodes[i].op == DVM_ISFINITE && e.cls[i] == CLS_TILE) flags |= DVM_F_EXT_ISA;
  for (int o = 0; o < p->n_outputs; ++o)  // a tile stored into a view whose rows are not one dense range: ViewStore
    if (e.cls[root(e, p->outputs[o].value)] == CLS_TILE && !dense_of[e.out_operand[o]]) flags |= DVM_F_VIEWS;
  for (int k = 0; k < e.n_in_regs; ++k)
    if (((best.lreg_table[k] >> 16) & 0xf) == DVM_LM_ROWS) flags |= DVM_F_LOADS_BY_ROW;
  for (int k = 0; k < e.n_in_regs; ++k)  // gathered rows: every thread fetches its own elements, in the views variant
    if (((best.lreg_table[k] >> 16) & 0xf) == DVM_LM_GATHER || ((best.lreg_table[k] >> 16) & 0xf) == DVM_LM_TRANSPOSED)
      flags |= DVM_F_LOADS_BY_ROW | DVM_F_VIEWS;

  // ---- 7. assemble ----
  const int n_tensors = n_in + p->n_outputs;
  const int code_words = e.n_loads + e.n_body;
  size_t words = DVM_HDR_WORDS + 2 * (size_t)n_tensors + (size_t)DVM_OPD_WORDS * e.n_opd + nreg + code_words;
  *code_size = words * 4;
  if (!code || code_capacity < words * 4) return DVM_ERR_BUFFER_TOO_SMALL;
  uint32_t* w = (uint32_t*)code;
  memset(w, 0, words * 4);
  w[DVM_H_MAGIC] = DVM_MAGIC;
  w[DVM_H_KERNEL_TYPE] = DVM_KERNEL_VEC;
  w[DVM_H_CODE_WORDS] = (uint32_t)code_words;
  w[DVM_H_N_TILES] = (uint32_t)n_tiles;
  w[DVM_H_TOTAL_WORDS] = (uint32_t)words;
  w[DVM_H_COUNTS] = (uint32_t)n_tensors | ((uint32_t)n_in << 8) | ((uint32_t)e.n_opd << 16) |
                    ((uint32_t)p->n_outputs << 24);
  w[DVM_H_GEOM] = (uint32_t)log2G | ((uint32_t)W << 8) | ((uint32_t)nreg << 16) | (flags << 24);
  w[DVM_H_COLS] = (uint32_t)C;
  w[DVM_H_ROWS_LO] = (uint32_t)rowsR;
  w[DVM_H_ROWS_HI] = (uint32_t)((uint64_t)rowsR >> 32);
  w[DVM_H_COL_BLOCKS] = (uint32_t)CB;
  w[DVM_H_COL_TILE] = (uint32_t)Ctile;
  w[DVM_H_OUTER0] = (uint32_t)outer[0];
  w[DVM_H_OUTER1] = (uint32_t)outer[1];
  w[DVM_H_OUTER2] = (uint32_t)outer[2];
  w[DVM_H_LAST_ROW_COLS] = (uint32_t)lastRowCols;
  w[DVM_H_PRIMARY] = primary >= 0 ? (uint32_t)primary : 0xffffffffu;
  w[DVM_H_LOCAL] = (uint32_t)e.n_in_regs | ((uint32_t)e.n_tmp_regs << 8) | ((uint32_t)e.n_sslots << 16) | ((uint32_t)best.V << 24);
  w[DVM_H_LOAD_WORDS] = (uint32_t)e.n_loads;
  w[DVM_H_LOCAL2] = (uint32_t)scalar_unit | ((uint32_t)units << 16);
  uint32_t* ot = w + DVM_HDR_WORDS + 2 * n_tensors;
  for (int o = 0; o < e.n_opd; ++o) {
    const Operand& od = e.opd[o];
    uint32_t* d = ot + o * DVM_OPD_WORDS;
    const bool dense = dense_of[o];
    d[DVM_OPD_INFO] = (uint32_t)od.slot | ((uint32_t)od.dtype << 8) | ((uint32_t)od.col_stride << 16) |
                      ((uint32_t)(od.primary ? 1 : 0) << 24) | ((uint32_t)(dense ? 1 : 0) << 25) |
                      ((uint32_t)od.combine << 26);
    d[DVM_OPD_COLSTRIDE] = (uint32_t)(uint64_t)od.cs;
    for (int g = 0; g < 3; ++g) {
      d[DVM_OPD_STRIDE0 + 2 * g] = (uint32_t)(uint64_t)od.ostride[g];
      d[DVM_OPD_STRIDE0 + 2 * g + 1] = (uint32_t)((uint64_t)od.ostride[g] >> 32);
    }
    if (od.combine) d[DVM_OPD_FILL] = (uint32_t)od.numel;  // (strides stay below 2^32: the word is free)
  }
  uint32_t* lt = ot + e.n_opd * DVM_OPD_WORDS;
  memcpy(lt, lreg_table, (size_t)nreg * 4);
  for (int q = 0; q < e.n_loads; ++q)
    if (DVM_INSN_OP(e.loads[q]) == DVM_OP_LDG && ((best.inv_mask >> DVM_INSN_A(e.loads[q])) & 1)) e.loads[q] |= 0x80u << 16;
  memcpy(lt + nreg, e.loads, (size_t)e.n_loads * 4);
  memcpy(lt + nreg + e.n_loads, e.body, (size_t)e.n_body * 4);
  if (C > 0xffffffffll || outer[0] > 0xffffffffll || outer[1] > 0xffffffffll || outer[2] > 0xffffffffll)
    return DVM_ERR_TOO_LARGE;
  for (int o = 0; o < e.n_opd; ++o)
    for (int q = 0; q < 3; ++q)
      if ((uint64_t)e.opd[o].ostride[q] > 0xffffffffull) return DVM_ERR_TOO_LARGE;  // the VM multiplies 32-bit strides
  for (int o = 0; o < e.n_opd; ++o)
    if ((uint64_t)e.opd[o].cs > 0xffffffffull || (uint64_t)e.opd[o].numel > 0xffffffffull) return DVM_ERR_TOO_LARGE;
  return DVM_OK;
}

static int encode_core(const dvm_program* p, const dvm_shape* in_shapes, const dvm_strides* in_strides, int n_in,
                       const float* scalars, int n_scalars, const dvm_strides* out_strides, void* code,
                       size_t code_capacity, size_t* code_size, dvm_shape* out_shapes, int n_out, bool lowered,
                       int combine_axis = 0) {
  if (!p || !in_shapes || !code_size) return DVM_ERR_INVALID_ARG;
  if (!p->finalized) return DVM_ERR_NOT_FINALIZED;
  if (n_in != p->n_inputs) return DVM_ERR_INVALID_ARG;
  if (n_scalars < p->n_params || (p->n_params > 0 && !scalars)) return DVM_ERR_INVALID_ARG;
  if (out_shapes && n_out < p->n_outputs) return DVM_ERR_INVALID_ARG;
  if (((uintptr_t)code & 7) != 0) return DVM_ERR_INVALID_ARG;
  if (p->n_matmul > 0) {
    if (in_strides || out_strides) return DVM_ERR_UNSUPPORTED;  // the matmul's tensor maps describe dense matrices
    return dvm_encode_matmul(p, in_shapes, n_in, scalars, n_scalars, code, code_capacity, code_size,
                             out_shapes, n_out);
  }

  Enc e;
  e.p = p;
  e.scalars = scalars;
  e.n_scalars = n_scalars;
  const int NN = p->n_nodes;

  // ---- 1. shape inference (numpy-style right-aligned broadcasting) ----
  int D = 1;
  for (int i = 0; i < n_in; ++i) {
    if (!lowered && in_shapes[i].rank != p->nodes[p->inputs[i]].rank) return DVM_ERR_INVALID_ARG;
    if (in_shapes[i].rank > D) D = in_shapes[i].rank;
  }
  {
    int ii = 0;
    for (int i = 0; i < NN; ++i) {
      const Node& n = p->nodes[i];
      int64_t* d = e.dims[i];
      e.alias[i] = -1;
      if (n.kind == NK_INPUT) {
        const dvm_shape& s = in_shapes[ii++];
        for (int k = 0; k < D; ++k) d[k] = 1;
        for (int k = 0; k < s.rank; ++k) {
          if (s.dims[k] < 0) return DVM_ERR_INVALID_ARG;
          d[D - s.rank + k] = s.dims[k];
        }
      } else if (n.kind == NK_BINARY || n.kind == NK_COMPARE || n.kind == NK_SELECT) {
        const int64_t* a = e.dims[n.x];
        const int64_t* b = e.dims[n.y];
        for (int k = 0; k < D; ++k) {
          if (a[k] == b[k]) d[k] = a[k];
          else if (a[k] == 1) d[k] = b[k];
          else if (b[k] == 1) d[k] = a[k];
          else return DVM_ERR_SHAPE_MISMATCH;
        }
        if (n.kind == NK_SELECT) {
          const int64_t* c3 = e.dims[n.param];
          for (int k = 0; k < D; ++k) {
            if (c3[k] == d[k] || c3[k] == 1) continue;
            if (d[k] == 1) d[k] = c3[k];
            else return DVM_ERR_SHAPE_MISMATCH;
          }
        }
      } else {
        for (int k = 0; k < D; ++k) d[k] = e.dims[n.x][k];
        if (n.kind == NK_REDUCE && !combine_axis) d[D - 1] = 1;
      }
    }
  }
  for (int k = 0; k < D; ++k) {
    int64_t m = 1;
    bool zero = false;
    for (int i = 0; i < NN; ++i) {
      if (e.dims[i][k] == 0) zero = true;
      if (e.dims[i][k] > m) m = e.dims[i][k];
    }
    e.Sd[k] = zero ? 0 : m;
  }
  for (int i = 0; i < NN; ++i)
    for (int k = 0; k < D; ++k)
      if (e.dims[i][k] != 1 && e.dims[i][k] != e.Sd[k]) return DVM_ERR_SHAPE_MISMATCH;
  if (out_shapes) {
    for (int o = 0; o < p->n_outputs; ++o) {
      // the rank of an output is the rank the dominant shape has (leading 1s kept)
      out_shapes[o].rank = D;
      for (int k = 0; k < DVM_MAX_RANK; ++k) out_shapes[o].dims[k] = k < D ? e.dims[p->outputs[o].value][k] : 0;
      if (combine_axis && p->nodes[p->outputs[o].value].kind == NK_REDUCE) out_shapes[o].dims[D + combine_axis] = 1;
    }
  }
  bool empty = false;
  for (int k = 0; k < D; ++k) if (e.Sd[k] == 0) empty = true;

  // ---- 2. classes: a value whose last dim is 1 while the dominant last dim is not is a per-row scalar ----
  int Dt = D;  // trailing size-1 dominant dims carry no extent: drop them
  while (Dt > 1 && e.Sd[Dt - 1] == 1) --Dt;
  const int64_t Ccols = e.Sd[Dt - 1] == 0 ? 1 : e.Sd[Dt - 1];  // (an instance without rows keeps its row length: classes as usual)
  bool has_reduce = false;
  for (int i = 0; i < NN; ++i) {
    const Node& n = p->nodes[i];
    int64_t last = e.dims[i][Dt - 1];
    e.cls[i] = (last == 1 && Ccols > 1) ? CLS_SCAL : CLS_TILE;
    if (n.kind == NK_REDUCE) {
      if (combine_axis || Dt < D || e.dims[n.x][Dt - 1] == 1) e.alias[i] = n.x;  // reducing a size-1 axis: identity
      else has_reduce = true;
    }
    if (n.kind == NK_CAST && n.dtype == DVM_F32) e.alias[i] = n.x;  // registers are fp32 already
  }

  // ---- 3. operands: inputs and outputs with their strides over the dominant dims ----
  e.n_opd = 0;
  int W = 4;
  for (int i = 0; i < n_in + p->n_outputs; ++i) {
    Operand& od = e.opd[e.n_opd];
    int v = i < n_in ? p->inputs[i] : p->outputs[i - n_in].value;
    od.slot = i;
    od.dtype = i < n_in ? p->nodes[v].dtype : p->outputs[i - n_in].dtype;
    od.primary = false;
    int64_t st = 1;
    for (int k = D - 1; k >= 0; --k) {
      int64_t dk = e.dims[v][k];
      od.stride[k] = (dk == 1 && e.Sd[k] != 1) ? 0 : st;
      st *= dk;
    }
    od.col_stride = (e.dims[v][Dt - 1] == 1 && Ccols > 1) ? 0 : 1;
    od.cs = 1;
    od.combine = 0;
    od.numel = 0;
    if (combine_axis && i >= n_in && p->nodes[v].kind == NK_REDUCE) {
      // the result of a reduction: dense over the reduced shape, stride 0 along the reduced axis
      if (out_strides || od.dtype != DVM_DT_F32) return DVM_ERR_UNSUPPORTED;
      const int q = D + combine_axis;
      int64_t s2 = 1;
      for (int k = D - 1; k >= 0; --k) {
        const int64_t dk = k == q ? 1 : e.dims[v][k];
        od.stride[k] = (k == q || (dk == 1 && e.Sd[k] != 1)) ? 0 : s2;
        s2 *= dk;
      }
      od.combine = 1 + p->nodes[v].op;
      od.numel = s2;
      if (q == Dt - 1) return DVM_ERR_UNSUPPORTED;  // (the reduced axis is never the column dim here)
    }
    const dvm_strides* us = i < n_in ? (in_strides ? &in_strides[i] : nullptr) : (out_strides ? &out_strides[i - n_in] : nullptr);
    if (us) {
      // a view: the caller's element strides replace the dense ones (dims of size 1 carry no stride)
      const int r = i < n_in ? in_shapes[i].rank : D;  // an output has the dominant rank
      for (int k = 0; k < D; ++k) {
        const int64_t dk = e.dims[v][k];
        const int uk = k - (D - r);
        if (dk == 1 || uk < 0) continue;
        const int64_t t = us->stride[uk];
        if (t < 0) return DVM_ERR_INVALID_ARG;
        if (i >= n_in && t == 0) return DVM_ERR_INVALID_ARG;  // a stored view addresses every element once
        od.stride[k] = t;
      }
      if (e.dims[v][Dt - 1] != 1) od.cs = od.stride[Dt - 1];  // != 1: the row's elements are gathered / scattered one by one
      if (i >= n_in) {
        // no two index tuples at one address: sorted by stride, each dim must step over the one before it
        int64_t sz[DVM_MAX_RANK], sd[DVM_MAX_RANK];
        int m = 0;
        for (int k = 0; k < D; ++k)
          if (e.dims[v][k] > 1) { sz[m] = e.dims[v][k]; sd[m] = od.stride[k]; ++m; }
        for (int a = 1; a < m; ++a)
          for (int b = a; b > 0 && sd[b] < sd[b - 1]; --b) { std::swap(sd[b], sd[b - 1]); std::swap(sz[b], sz[b - 1]); }
        for (int a = 1; a < m; ++a)
          if (sd[a] < sd[a - 1] * sz[a - 1]) return DVM_ERR_INVALID_ARG;
      }
    }
    if (i >= n_in) {
      // an output must cover the dominant shape (or be one value per row); otherwise several
      // tiles would write the same element
      for (int k = 0; k < Dt - 1; ++k)
        if (e.dims[v][k] != e.Sd[k]) return DVM_ERR_UNSUPPORTED;
      e.out_operand[i - n_in] = (int8_t)e.n_opd;
    } else {
      e.in_operand[v] = (int8_t)e.n_opd;
    }
    if (od.col_stride == 1 && od.cs == 1 && od.dtype == DVM_DT_BF16) W = 8;
    e.n_opd++;
  }

  // ---- 4. merge adjacent dims that are dense in every operand (dims of size 1 vanish) ----
  // groups are collected innermost first; group 0 is the column dim.
  int64_t gsize[DVM_MAX_RANK];
  int64_t gstride[DVM_MAX_OPERANDS][DVM_MAX_RANK];
  int ng = 0;
  for (int k = Dt - 1; k >= 0; --k) {
    if (e.Sd[k] == 1 && k != Dt - 1) continue;
    bool merged = ng > 0 && !(ng == 1 && has_reduce);  // a reduced row never merges with outer dims
    if (merged) {
      for (int o = 0; o < e.n_opd; ++o)
        if (e.opd[o].stride[k] != gstride[o][ng - 1] * gsize[ng - 1]) { merged = false; break; }
    }
    if (merged) {
      gsize[ng - 1] *= e.Sd[k];
    } else {
      gsize[ng] = e.Sd[k];
      for (int o = 0; o < e.n_opd; ++o) gstride[o][ng] = (k == Dt - 1) ? (e.opd[o].col_stride ? e.opd[o].cs : 0) : e.opd[o].stride[k];
      ng++;
    }
  }
  if (ng > 4) return DVM_ERR_UNSUPPORTED;
  int64_t C = gsize[0];
  int64_t outer[3] = {1, 1, 1};
  for (int g = 1; g < ng; ++g) outer[g - 1] = gsize[g];
  for (int o = 0; o < e.n_opd; ++o)
    for (int g = 0; g < 3; ++g) e.opd[o].ostride[g] = (g + 1 < ng) ? gstride[o][g + 1] : 0;
  int64_t R = outer[0] * outer[1] * outer[2];
  if (empty) { R = 0; C = 1; }
  const bool flat = (ng == 1) && !has_reduce;

  // primary operand: the first tile-class access that spans the whole dominant shape
  int primary = -1;
  for (int o = 0; o < e.n_opd && primary < 0; ++o) {
    const Operand& od = e.opd[o];
    if (od.col_stride != 1 || od.cs != 1 || od.dtype > DVM_DT_BF16) continue;  // (never an integer output: the chunks follow 2- or 4-byte elements)
    bool full = true;
    for (int g = 0; g < 3; ++g) if (outer[g] > 1 && od.ostride[g] == 0) full = false;
    if (full) primary = o;
  }
  if (primary < 0) {
    for (int o = 0; o < e.n_opd && primary < 0; ++o)
      if (e.opd[o].col_stride == 1 && e.opd[o].cs == 1 && e.opd[o].dtype <= DVM_DT_BF16) primary = o;
  }
  // combined results: the rows a warp holds are combined slot by slot, so every row must map its columns to
  // the same slots -- no operand to align the chunks to, every operand is read at its own phase
  if (combine_axis) primary = -1;
  if (primary >= 0) e.opd[primary].primary = true;

  // ---- 5. code: load section + compute section (independent of the tile geometry) ----
  // a reduced row longer than the widest tile (256 threads x 32 elements) is walked in column blocks, in phases
  e.phased = has_reduce && !combine_axis && !empty && C > (int64_t)DVM_VM_THREADS * DVM_VM_VMAX;
  e.n_phases = 1;
  if (!gen_body(e)) return DVM_ERR_UNSUPPORTED;  // more live tile values than local registers
  if (e.phased && !tag_phases(e)) return DVM_ERR_UNSUPPORTED;  // more phases, or per-row scalars, than the machine holds
  const int nreg = e.n_in_regs + e.n_tmp_regs;
  int in_dtype[DVM_MAX_LREGS], in_opd[DVM_MAX_LREGS];
  for (int k = 0; k < e.n_in_regs; ++k) {
    in_dtype[k] = DVM_DT_F32;
    in_opd[k] = 0;
    for (int q = 0; q < e.n_loads; ++q)
      if (DVM_INSN_OP(e.loads[q]) == DVM_OP_LDG && (int)DVM_INSN_A(e.loads[q]) == k) {
        in_opd[k] = (int)DVM_INSN_B(e.loads[q]);
        in_dtype[k] = e.opd[in_opd[k]].dtype;
      }
  }

  // ---- 6. shape tiling, 7. assembly ----
  Lowered L;
  L.C = C; L.R = R;
  for (int q = 0; q < 3; ++q) L.outer[q] = outer[q];
  L.flat = flat; L.empty = empty; L.has_reduce = has_reduce;
  L.primary = primary; L.combine_axis = combine_axis; L.W = W; L.nreg = nreg;
  for (int k = 0; k < DVM_MAX_LREGS; ++k) { L.in_dtype[k] = k < e.n_in_regs ? in_dtype[k] : 0; L.in_opd[k] = k < e.n_in_regs ? in_opd[k] : 0; }
  Geo best;
  const int gst = choose_geometry(e, L, best);
  if (gst != DVM_OK) return gst;
  return assemble_program(e, L, best, n_in, code, code_capacity, code_size);
}

// Reductions over another axis than the last (Table 1, Sum / Max / Min of [M, size, N] over `size`) are lowered
// to views: elementwise operators do not care in which order the dims are walked, so the reduced axis is moved
// to the end for EVERY operand (shapes and element strides permuted alike), the program is encoded as a
// last-axis reduction over those views (ViewLoad / ViewStore), and the reported output shapes are permuted back.
static int encode_views(const dvm_program* p, const dvm_shape* in_shapes, const dvm_strides* in_strides, int n_in,
                        const float* scalars, int n_scalars, const dvm_strides* out_strides, void* code,
                        size_t code_capacity, size_t* code_size, dvm_shape* out_shapes, int n_out) {
  if (!p || !in_shapes || !code_size) return DVM_ERR_INVALID_ARG;
  if (!p->finalized) return DVM_ERR_NOT_FINALIZED;
  int ax = -1;
  bool last_too = false;
  for (int i = 0; i < p->n_nodes; ++i) {
    if (p->nodes[i].kind != NK_REDUCE) continue;
    const int a = p->nodes[i].param;
    if (a == -1) { last_too = true; continue; }
    if (ax != -1 && ax != a) return DVM_ERR_UNSUPPORTED;  // one reduced axis per program
    ax = a;
  }
  if (ax == -1)
    return encode_core(p, in_shapes, in_strides, n_in, scalars, n_scalars, out_strides, code, code_capacity, code_size,
                       out_shapes, n_out, false);
  if (last_too || p->n_matmul > 0) return DVM_ERR_UNSUPPORTED;
  if (n_in != p->n_inputs) return DVM_ERR_INVALID_ARG;
  {
    int rank = 1;
    for (int i = 0; i < n_in; ++i) {
      if (in_shapes[i].rank != p->nodes[p->inputs[i]].rank || in_shapes[i].rank > DVM_MAX_RANK) return DVM_ERR_INVALID_ARG;
      if (in_shapes[i].rank > rank) rank = in_shapes[i].rank;
    }
    if (-ax > rank) return DVM_ERR_INVALID_ARG;  // no such axis
  }
  // Reductions that are results only (nothing in the program reads them), stored as fp32, dense: no view, no
  // gather -- the program runs over its natural tiles (columns adjacent in memory) and every tile combines
  // its rows into the result with atomic operations.
  {
    bool results_only = !out_strides;
    for (int i = 0; i < p->n_nodes && results_only; ++i) {
      const Node& n = p->nodes[i];
      const int ops[3] = {n.kind == NK_INPUT ? -1 : n.x,
                          (n.kind == NK_BINARY || n.kind == NK_COMPARE || n.kind == NK_SELECT) ? n.y : -1,
                          n.kind == NK_SELECT ? n.param : -1};
      for (int k = 0; k < 3; ++k)
        if (ops[k] >= 0 && p->nodes[ops[k]].kind == NK_REDUCE) results_only = false;
    }
    for (int o = 0; o < p->n_outputs && results_only; ++o)
      if (p->nodes[p->outputs[o].value].kind == NK_REDUCE && p->outputs[o].dtype != DVM_F32) results_only = false;
    if (results_only) {
      int st = encode_core(p, in_shapes, in_strides, n_in, scalars, n_scalars, nullptr, code, code_capacity, code_size,
                           out_shapes, n_out, false, ax);
      if (st != DVM_ERR_UNSUPPORTED) return st;  // otherwise (e.g. the reduced axis ends up as the column dim): the view lowering
    }
  }
  if (n_in != p->n_inputs || n_in > DVM_MAX_TENSORS || p->n_outputs > DVM_MAX_TENSORS) return DVM_ERR_INVALID_ARG;
  int D = 1;
  for (int i = 0; i < n_in; ++i) {
    if (in_shapes[i].rank != p->nodes[p->inputs[i]].rank || in_shapes[i].rank > DVM_MAX_RANK) return DVM_ERR_INVALID_ARG;
    if (in_shapes[i].rank > D) D = in_shapes[i].rank;
  }
  if (-ax > D) return DVM_ERR_INVALID_ARG;  // no such axis
  const int q = D + ax;                      // the reduced dim of the right-aligned dominant shape
  int perm[DVM_MAX_RANK];                    // dim k of the permuted shape is dim perm[k] of the original
  for (int k = 0, m = 0; k < D; ++k)
    if (k != q) perm[m++] = k;
  perm[D - 1] = q;
  dvm_shape ps[DVM_MAX_TENSORS];
  dvm_strides pst[DVM_MAX_TENSORS];
  for (int i = 0; i < n_in; ++i) {
    const int r = in_shapes[i].rank;
    int64_t d[DVM_MAX_RANK], t[DVM_MAX_RANK];
    int64_t st = 1;
    for (int k = D - 1; k >= 0; --k) {
      const int uk = k - (D - r);
      d[k] = uk >= 0 ? in_shapes[i].dims[uk] : 1;
      t[k] = uk >= 0 ? (in_strides ? in_strides[i].stride[uk] : st) : 0;
      if (d[k] < 0) return DVM_ERR_INVALID_ARG;
      st *= d[k] > 0 ? d[k] : 1;
    }
    ps[i].rank = D;
    for (int k = 0; k < DVM_MAX_RANK; ++k) { ps[i].dims[k] = k < D ? d[perm[k]] : 0; pst[i].stride[k] = k < D ? t[perm[k]] : 0; }
  }
  // pass 1: the output shapes (in permuted order); pass 2: with the outputs' strides permuted as well
  dvm_shape pos[DVM_MAX_TENSORS];
  int st = encode_core(p, ps, pst, n_in, scalars, n_scalars, nullptr, code, code_capacity, code_size, pos, p->n_outputs, true);
  if (st != DVM_OK) return st;
  dvm_strides post[DVM_MAX_TENSORS];
  for (int o = 0; o < p->n_outputs; ++o) {
    int64_t d[DVM_MAX_RANK], t[DVM_MAX_RANK];
    for (int k = 0; k < D; ++k) d[perm[k]] = pos[o].dims[k];  // back to the caller's order
    int64_t s2 = 1;
    for (int k = D - 1; k >= 0; --k) {
      t[k] = out_strides ? out_strides[o].stride[k] : s2;
      s2 *= d[k] > 0 ? d[k] : 1;
    }
    for (int k = 0; k < DVM_MAX_RANK; ++k) post[o].stride[k] = k < D ? t[perm[k]] : 0;
    if (out_shapes && o < n_out) {
      out_shapes[o].rank = D;
      for (int k = 0; k < DVM_MAX_RANK; ++k) out_shapes[o].dims[k] = k < D ? d[k] : 0;
    }
  }
  if (out_shapes && n_out < p->n_outputs) return DVM_ERR_INVALID_ARG;
  return encode_core(p, ps, pst, n_in, scalars, n_scalars, post, code, code_capacity, code_size, nullptr, 0, true);
}

extern "C" int dvm_encode(const dvm_program* p, const dvm_shape* in_shapes, int n_in,
                          const float* scalars, int n_scalars, void* code, size_t code_capacity,
                          size_t* code_size, dvm_shape* out_shapes, int n_out) {
  return encode_views(p, in_shapes, nullptr, n_in, scalars, n_scalars, nullptr, code, code_capacity, code_size,
                      out_shapes, n_out);
}

extern "C" int dvm_encode_strided(const dvm_program* p, const dvm_shape* in_shapes, const dvm_strides* in_strides,
                                  int n_in, const float* scalars, int n_scalars, const dvm_strides* out_strides,
                                  void* code, size_t code_capacity, size_t* code_size, dvm_shape* out_shapes,
                                  int n_out) {
  return encode_views(p, in_shapes, in_strides, n_in, scalars, n_scalars, out_strides, code, code_capacity,
                      code_size, out_shapes, n_out);
}

extern "C" int dvm_time_encode(const dvm_program* p, const dvm_shape* in_shapes, const dvm_strides* in_strides, int n_in,
                               const float* scalars, int n_scalars, void* code, size_t code_capacity, int reps,
                               int64_t* ns_out) {
  if (reps < 0 || (reps > 0 && !ns_out)) return DVM_ERR_INVALID_ARG;
  for (int r = 0; r < reps; ++r) {
    size_t size = 0;
    const auto t0 = std::chrono::steady_clock::now();
    const int st = encode_views(p, in_shapes, in_strides, n_in, scalars, n_scalars, nullptr, code, code_capacity, &size,
                                nullptr, 0);
    const auto t1 = std::chrono::steady_clock::now();
    if (st != DVM_OK) return st;
    ns_out[r] = (int64_t)std::chrono::duration_cast<std::chrono::nanoseconds>(t1 - t0).count();
  }
  return DVM_OK;
}

extern "C" int dvm_encode_batch(int n, const dvm_program* const* programs, const dvm_shape* in_shapes, const int* n_in,
                                const float* scalars, const int* n_scalars, void* const* codes, const size_t* caps,
                                size_t* sizes, int* failed) {
  if (n < 0 || (n > 0 && (!programs || !in_shapes || !n_in || !n_scalars || !codes || !caps || !sizes)))
    return DVM_ERR_INVALID_ARG;
  size_t si = 0, fi = 0;
  for (int i = 0; i < n; ++i) {
    if (n_in[i] < 0 || n_scalars[i] < 0) {
      if (failed) *failed = i;
      return DVM_ERR_INVALID_ARG;
    }
    const int st = dvm_encode(programs[i], in_shapes + si, n_in[i], n_scalars[i] ? scalars + fi : nullptr, n_scalars[i],
                              codes[i], caps[i], &sizes[i], nullptr, 0);
    if (st != DVM_OK) {
      if (failed) *failed = i;
      return st;
    }
    si += (size_t)n_in[i];
    fi += (size_t)n_scalars[i];
  }
  return DVM_OK;
}

// ---------------------------------------------------------------------------
// Verification and the readable dump
// ---------------------------------------------------------------------------
static int insn_expected_len(uint32_t op, uint32_t w0) {
  if (op <= DVM_OP_BCS || op == DVM_OP_PHASE) return 1;
  if (op == DVM_OP_SOP) return DVM_INSN_B(w0) == DVM_SK_BINI ? 3 : (DVM_INSN_B(w0) == DVM_SK_FMAU ? 4 : 2);
  if (op >= DVM_OP_LD2 && op < DVM_OP_LD2 + DVM_A_NBIN) return 1;
  if (op >= DVM_OP_CMP && op < DVM_OP_CMP + DVM_C_NCMP) return 1;
  if (op >= DVM_OP_SEL && op < DVM_OP_SEL + 3) return 1;
  if (op == DVM_OP_SEL + 3) return 3;
  if (op >= DVM_OP_BINI && op < DVM_OP_BINI + DVM_A_NBIN) return 2;
  if (op >= DVM_OP_BIN && op < DVM_OP_BIN + DVM_A_NBIN) return 1;
  if (op >= DVM_OP_BINS && op < DVM_OP_BINS + DVM_A_NBIN) return 1;
  if (op >= DVM_OP_UN && op < DVM_OP_UN + DVM_U_NUN) return 1;
  if (op >= DVM_OP_ACT && op < DVM_OP_ACT + DVM_ACT_N) return 1;
  if (op >= DVM_OP_RED && op < DVM_OP_RED + DVM_R_NRED) return 1;
  if (op == DVM_OP_SOP) return DVM_INSN_B(w0) == DVM_SK_BINI ? 3 : 2;
  return -1;
}

int dvm_verify_matmul(const uint32_t* w, size_t n_words);

extern "C" int dvm_verify(const void* code, size_t code_size) {
  if (!code) return DVM_ERR_INVALID_ARG;
  if (code_size < DVM_HDR_WORDS * 4 || (code_size & 3) || ((uintptr_t)code & 3)) return DVM_ERR_BAD_CODE;
  const uint32_t* w = (const uint32_t*)code;
  if (w[DVM_H_MAGIC] != DVM_MAGIC) return DVM_ERR_BAD_CODE;
  if (w[DVM_H_TOTAL_WORDS] * 4ull != code_size) return DVM_ERR_BAD_CODE;
  if (w[DVM_H_KERNEL_TYPE] == DVM_KERNEL_MATMUL) return dvm_verify_matmul(w, code_size / 4);
  if (w[DVM_H_KERNEL_TYPE] != DVM_KERNEL_VEC) return DVM_ERR_BAD_CODE;
  uint32_t counts = w[DVM_H_COUNTS];
  uint32_t n_tensors = counts & 0xff, n_in = (counts >> 8) & 0xff, n_opd = (counts >> 16) & 0xff,
           n_out = counts >> 24;
  if (n_tensors > DVM_MAX_TENSORS || n_opd > DVM_MAX_OPERANDS || n_in + n_out != n_tensors) return DVM_ERR_BAD_CODE;
  uint32_t body = w[DVM_H_CODE_WORDS];
  const uint32_t n_lregs = (w[DVM_H_GEOM] >> 16) & 0xff;
  if ((uint64_t)DVM_HDR_WORDS + 2 * n_tensors + DVM_OPD_WORDS * n_opd + n_lregs + body != w[DVM_H_TOTAL_WORDS])
    return DVM_ERR_BAD_CODE;
  uint32_t geom = w[DVM_H_GEOM];
  uint32_t lg = geom & 0xff, W = (geom >> 8) & 0xff, nreg = (geom >> 16) & 0xff;
  const uint32_t local = w[DVM_H_LOCAL];
  const uint32_t n_inr = local & 0xff, n_tmpr = (local >> 8) & 0xff, n_ss = (local >> 16) & 0xff, Vv = local >> 24;
  if (Vv != 16 && Vv != 24 && Vv != 32) return DVM_ERR_BAD_CODE;
  const uint32_t u_bf16 = DVM_DT_BF16, u_f32 = DVM_DT_F32;  // element type an instruction expects in a register
  if (lg > 8 || !(W == 4 || W == 8) || nreg != n_inr + n_tmpr) return DVM_ERR_BAD_CODE;
  const uint32_t local2 = w[DVM_H_LOCAL2];
  const uint32_t units = local2 >> 16, scalar_unit = local2 & 0xffffu;
  if (n_inr + n_tmpr > DVM_MAX_LREGS || n_ss > DVM_MAX_SSLOTS || 2 * units + 1 > DVM_MAX_LOCAL_UNITS) return DVM_ERR_BAD_CODE;
  if (n_ss && scalar_unit + 2 * 16 * DVM_VM_THREADS / DVM_LOCAL_UNIT > units) return DVM_ERR_BAD_CODE;
  const uint32_t* lt = w + DVM_HDR_WORDS + 2 * n_tensors + DVM_OPD_WORDS * n_opd;
  const uint32_t* otab = w + DVM_HDR_WORDS + 2 * n_tensors;
  // a local register must lie inside the tile slot, in the layout its kind implies, and hold the element
  // type the instruction expects
  auto lreg_ok = [&](uint32_t k, uint32_t dt) {
    if (k >= nreg) return false;
    const uint32_t lw = lt[k], unit = lw & 0xffffu, mode = (lw >> 16) & 0xff, od = lw >> 24;  // bits 20..23 (address phase) are set at launch only
    uint64_t need;
    if (k >= n_inr) {
      if (mode != DVM_LM_PRIVATE || dt != DVM_DT_F32) return false;
      need = (uint64_t)Vv * 4 * DVM_VM_THREADS / DVM_LOCAL_UNIT;
    } else if (mode == DVM_LM_GATHER) {
      if (od >= n_opd || dt != DVM_DT_F32 || !((w[DVM_H_GEOM] >> 24) & DVM_F_VIEWS)) return false;
      need = (uint64_t)Vv * 4 * DVM_VM_THREADS / DVM_LOCAL_UNIT;
    } else if (mode == DVM_LM_TRANSPOSED) {
      // one strip per column of the column block, each holding the tile's rows: at most one strip per thread,
      // strips and column stride in whole 16-byte units, rows adjacent in memory
      if (od >= n_opd || dt != DVM_DT_F32 || !((w[DVM_H_GEOM] >> 24) & DVM_F_VIEWS)) return false;
      const uint32_t* d = otab + od * DVM_OPD_WORDS;
      const uint64_t es = 1ull << DVM_DT_LG_ES((d[0] >> 8) & 0xff), Rt = DVM_VM_THREADS >> lg;
      if (((uint64_t)Vv << lg) > DVM_VM_THREADS || (Rt * es) % 16 || ((uint64_t)d[DVM_OPD_COLSTRIDE] * es) % 16 || d[DVM_OPD_STRIDE0] != 1 ||
          (w[DVM_H_GEOM] >> 24) & DVM_F_FLAT)
        return false;
      if ((w[DVM_H_OUTER1] > 1 || w[DVM_H_OUTER2] > 1) &&
          (((uint64_t)d[DVM_OPD_STRIDE1] * es) % 16 || ((uint64_t)d[DVM_OPD_STRIDE2] * es) % 16 || w[DVM_H_OUTER0] % Rt))
        return false;
      need = ((uint64_t)w[DVM_H_COL_TILE] * DVM_STRIP_PITCH(Rt, es) + DVM_LOCAL_UNIT - 1) / DVM_LOCAL_UNIT;
    } else {
      if (mode < DVM_LM_BLOCK || mode > DVM_LM_BCAST_TILE || od >= n_opd) return false;
      if (mode == DVM_LM_BCAST && w[DVM_H_COL_BLOCKS] > 1) return false;  // a once-per-program image holds whole rows
      if (((otab[od * DVM_OPD_WORDS] >> 8) & 0xff) != dt) return false;
      const uint64_t pitch = DVM_ROW_PITCH(1u << lg, Vv, dt == DVM_DT_BF16 ? 2 : 4);
      const uint64_t bytes = mode >= DVM_LM_BCAST ? pitch : pitch * (DVM_VM_THREADS >> lg);
      need = (bytes + DVM_LOCAL_UNIT - 1) / DVM_LOCAL_UNIT;
    }
    return unit + need <= units;
  };
  const uint32_t load_words = w[DVM_H_LOAD_WORDS];
  if (load_words > body) return DVM_ERR_BAD_CODE;
  uint64_t G = 1ull << lg;
  uint64_t ctile = w[DVM_H_COL_TILE], cb = w[DVM_H_COL_BLOCKS], C = w[DVM_H_COLS];
  uint64_t R = (uint64_t)w[DVM_H_ROWS_LO] | ((uint64_t)w[DVM_H_ROWS_HI] << 32);
  uint32_t flags = geom >> 24;
  const uint64_t pad = 0;  // a misaligned row that fills the whole capacity wraps its last columns into the head slots
  // a phased program (rows longer than a tile) says so in the first word of its compute section
  const uint32_t n_phases = load_words < body ? DVM_PHASES_OF((lt + n_lregs)[load_words]) : 0u;  // 0: not phased
  if (n_phases > DVM_MAX_PHASES) return DVM_ERR_BAD_CODE;
  if (n_phases && (lg != 8 || (flags & DVM_F_FLAT))) return DVM_ERR_BAD_CODE;  // one row per tile
  if (!(flags & DVM_F_ALIGNED) && w[DVM_H_PRIMARY] == 0xffffffffu) return DVM_ERR_BAD_CODE;
  if (w[DVM_H_N_TILES] > 0) {
    if (ctile == 0 || cb == 0 || ctile + pad > G * Vv) return DVM_ERR_BAD_CODE;
    if (cb * ctile < C || (cb - 1) * ctile >= C) return DVM_ERR_BAD_CODE;
    uint64_t rpt = DVM_VM_THREADS / G;
    if ((uint64_t)w[DVM_H_N_TILES] != ((R + rpt - 1) / rpt) * cb * (n_phases ? n_phases : 1u)) return DVM_ERR_BAD_CODE;
    if (w[DVM_H_LAST_ROW_COLS] == 0 || w[DVM_H_LAST_ROW_COLS] > C) return DVM_ERR_BAD_CODE;
    if ((uint64_t)w[DVM_H_OUTER0] * w[DVM_H_OUTER1] * w[DVM_H_OUTER2] != R) return DVM_ERR_BAD_CODE;
  }
  const uint32_t* ot = w + DVM_HDR_WORDS + 2 * n_tensors;
  int n_primary = 0;
  for (uint32_t o = 0; o < n_opd; ++o) {
    uint32_t info = ot[o * DVM_OPD_WORDS + DVM_OPD_INFO];
    if ((info & 0xff) >= n_tensors) return DVM_ERR_BAD_CODE;
    if (((info >> 8) & 0xff) > (uint32_t)((info & 0xff) < n_in ? DVM_DT_BF16 : DVM_DT_I32)) return DVM_ERR_BAD_CODE;  // integer types: outputs only
    if (((info >> 24) & 1) && ((info >> 8) & 0xff) > DVM_DT_BF16) return DVM_ERR_BAD_CODE;                            // ... and never the primary operand
    if (((info >> 16) & 0xff) > 1) return DVM_ERR_BAD_CODE;
    const uint32_t combine = (info >> 26) & 3;
    if (ot[o * DVM_OPD_WORDS + 3] | ot[o * DVM_OPD_WORDS + 5]) return DVM_ERR_BAD_CODE;  // 32-bit strides
    if (!combine && ot[o * DVM_OPD_WORDS + DVM_OPD_FILL]) return DVM_ERR_BAD_CODE;
    n_primary += (info >> 24) & 1;
    if (info >> 28) return DVM_ERR_BAD_CODE;
    if (combine) {
      // an fp32 result that tiles combine atomically: an output, run by the views variant, never "dense"
      if ((info & 0xff) < n_in || ((info >> 8) & 0xff) != DVM_DT_F32 || ((info >> 25) & 1) || ((info >> 24) & 1) ||
          !((w[DVM_H_GEOM] >> 24) & DVM_F_VIEWS) || (w[DVM_H_GEOM] & 0xff) > 5)
        return DVM_ERR_BAD_CODE;
    }
  }
  if (n_primary > 1) return DVM_ERR_BAD_CODE;
  if (w[DVM_H_PRIMARY] != 0xffffffffu) {
    if (w[DVM_H_PRIMARY] >= n_opd || !((ot[w[DVM_H_PRIMARY] * DVM_OPD_WORDS] >> 24) & 1)) return DVM_ERR_BAD_CODE;
  } else if (n_primary != 0) {
    return DVM_ERR_BAD_CODE;
  }
  const uint32_t* b = ot + n_opd * DVM_OPD_WORDS + n_lregs;
  uint32_t pc = 0;
  while (pc < body) {
    uint32_t w0 = b[pc], op = DVM_INSN_OP(w0), len = DVM_INSN_LEN(w0), a = DVM_INSN_A(w0), bb = DVM_INSN_B(w0);
    int el = insn_expected_len(op, w0);
    if (el < 0 || (uint32_t)el != len || pc + len > body) return DVM_ERR_BAD_CODE;
    const bool in_load = pc < load_words;
    if ((op == DVM_OP_LDG || op == DVM_OP_LDS) != in_load) return DVM_ERR_BAD_CODE;  // loads live in the load section only
    {
      // phase tags: on the run-once instructions of a phased program only
      const uint32_t tag = DVM_INSN_TAG(w0);
      const bool taggable = op == DVM_OP_STG || op == DVM_OP_STS || op == DVM_OP_SOP || (op >= DVM_OP_RED && op < DVM_OP_RED + DVM_R_NRED);
      if (tag > (taggable ? n_phases : 0u)) return DVM_ERR_BAD_CODE;
      if (n_phases && tag == 0 && (op == DVM_OP_STG || op == DVM_OP_STS || (op >= DVM_OP_RED && op < DVM_OP_RED + DVM_R_NRED)))
        return DVM_ERR_BAD_CODE;
      if (op == DVM_OP_PHASE) {
        if (pc == load_words ? (a != 0xffu || bb < 1) : (a < 1 || a >= n_phases || bb != 0)) return DVM_ERR_BAD_CODE;
      }
    }
    if (op == DVM_OP_LDG || op == DVM_OP_STG) {
      if (bb >= n_opd) return DVM_ERR_BAD_CODE;
      uint32_t info = ot[bb * DVM_OPD_WORDS];
      if (op == DVM_OP_LDG) {
        if ((a & 0x7f) >= n_inr) return DVM_ERR_BAD_CODE;
        const uint32_t lmode = (lt[a & 0x7f] >> 16) & 0xff;
        const bool gathered = lmode == DVM_LM_GATHER || lmode == DVM_LM_TRANSPOSED;  // read as fp32 by the instructions
        if (!lreg_ok(a & 0x7f, (!gathered && ((info >> 8) & 0xff) == DVM_DT_BF16) ? u_bf16 : u_f32)) return DVM_ERR_BAD_CODE;
        if (gathered != (ot[bb * DVM_OPD_WORDS + DVM_OPD_COLSTRIDE] != 1)) return DVM_ERR_BAD_CODE;
      }
      bool is_out = (info & 0xff) >= n_in;
      if ((op == DVM_OP_STG) != is_out) return DVM_ERR_BAD_CODE;  // never store to an input, never load an output
      if (((info >> 16) & 0xff) != 1) return DVM_ERR_BAD_CODE;
    } else if (op == DVM_OP_LDS || op == DVM_OP_STS) {
      if (bb >= n_opd) return DVM_ERR_BAD_CODE;
      if (op == DVM_OP_LDS ? a >= n_ss : a >= DVM_MAX_SREGS) return DVM_ERR_BAD_CODE;
      uint32_t info = ot[bb * DVM_OPD_WORDS];
      bool is_out = (info & 0xff) >= n_in;
      if ((op == DVM_OP_STS) != is_out) return DVM_ERR_BAD_CODE;
      if (((info >> 16) & 0xff) != 0) return DVM_ERR_BAD_CODE;
    } else if (op == DVM_OP_LDA) {
      if (bb > DVM_DT_BF16 || !lreg_ok(a, bb == DVM_DT_BF16 ? u_bf16 : u_f32)) return DVM_ERR_BAD_CODE;
    } else if (op == DVM_OP_STA) {
      if (a < n_inr || !lreg_ok(a, u_f32)) return DVM_ERR_BAD_CODE;  // input registers are read-only
    } else if (op == DVM_OP_LSS) {
      if (a >= DVM_MAX_SREGS || bb >= n_ss) return DVM_ERR_BAD_CODE;
    } else if (op == DVM_OP_BCS) {
      if (a >= DVM_MAX_SREGS) return DVM_ERR_BAD_CODE;
    } else if (op >= DVM_OP_BIN && op < DVM_OP_BIN + DVM_A_NBIN) {
      if (bb > DVM_DT_BF16 || (a != DVM_REG_ACC && !lreg_ok(a, bb == DVM_DT_BF16 ? u_bf16 : u_f32))) return DVM_ERR_BAD_CODE;
    } else if ((op >= DVM_OP_BINS && op < DVM_OP_BINS + DVM_A_NBIN) ||
               (op >= DVM_OP_RED && op < DVM_OP_RED + DVM_R_NRED)) {
      if (a >= DVM_MAX_SREGS) return DVM_ERR_BAD_CODE;
    } else if (op == DVM_OP_SOP) {
      uint32_t w1 = b[pc + 1], sub = w1 & 0xff, s1 = (w1 >> 8) & 0xff, s2 = (w1 >> 16) & 0xff;
      if (a >= DVM_MAX_SREGS || s1 >= DVM_MAX_SREGS) return DVM_ERR_BAD_CODE;
      if (bb == DVM_SK_BIN) { if (sub >= DVM_A_NBIN || s2 >= DVM_MAX_SREGS) return DVM_ERR_BAD_CODE; }
      else if (bb == DVM_SK_BINI) { if (sub >= DVM_A_NBIN) return DVM_ERR_BAD_CODE; }
      else if (bb == DVM_SK_UN) { if (sub >= DVM_U_NUN) return DVM_ERR_BAD_CODE; }
      else if (bb == DVM_SK_FMAU) { if (sub >= DVM_U_NUN && sub != 0xff) return DVM_ERR_BAD_CODE; }
      else return DVM_ERR_BAD_CODE;
    } else if ((op >= DVM_OP_LD2 && op < DVM_OP_LD2 + DVM_A_NBIN) || (op >= DVM_OP_SEL && op < DVM_OP_SEL + 3)) {
      if (!lreg_ok(a, ((bb >> 6) & 1) ? u_bf16 : u_f32) || !lreg_ok(bb & 0x3f, (bb >> 7) ? u_bf16 : u_f32)) return DVM_ERR_BAD_CODE;
    } else if (op >= DVM_OP_CMP && op < DVM_OP_CMP + DVM_C_NCMP) {
      if (bb > DVM_DT_BF16 || (a != DVM_REG_ACC && !lreg_ok(a, bb == DVM_DT_BF16 ? u_bf16 : u_f32))) return DVM_ERR_BAD_CODE;
    }
    pc += len;
  }
  return pc == body ? DVM_OK : DVM_ERR_BAD_CODE;
}

namespace {
struct Out {
  char* buf;
  size_t cap, len;
  bool overflow;
};
static void outf(Out& o, const char* fmt, ...) {
  char tmp[256];
  va_list ap;
  va_start(ap, fmt);
  int n = vsnprintf(tmp, sizeof tmp, fmt, ap);
  va_end(ap);
  if (n < 0) return;
  if ((size_t)n >= sizeof tmp) n = sizeof tmp - 1;
  if (o.len + (size_t)n + 1 > o.cap) { o.overflow = true; return; }
  memcpy(o.buf + o.len, tmp, (size_t)n);
  o.len += (size_t)n;
  o.buf[o.len] = 0;
}
static const char* kArith[8] = {"add", "sub", "rsub", "mul", "div", "rdiv", "min", "max"};
static const char* kUn[DVM_U_NUN] = {"exp", "sqrt", "rsqrt", "abs", "log", "erf", "sigmoid", "neg",
                                     "recip", "floor", "round", "tanh", "rnd_bf16", "isfinite", "trunc_i32", "trunc_u8"};
static const char* kRed[DVM_R_NRED] = {"sum", "max", "min", "sumsq"};
}  // namespace

int dvm_disassemble_matmul(const uint32_t* w, size_t n_words, char* buf, size_t cap);

extern "C" int dvm_disassemble(const void* code, size_t code_size, char* buf, size_t cap) {
  if (!buf || cap == 0) return DVM_ERR_INVALID_ARG;
  buf[0] = 0;
  int st = dvm_verify(code, code_size);
  if (st != DVM_OK) return st;
  const uint32_t* w = (const uint32_t*)code;
  if (w[DVM_H_KERNEL_TYPE] == DVM_KERNEL_MATMUL) return dvm_disassemble_matmul(w, code_size / 4, buf, cap);
  Out o = {buf, cap, 0, false};
  uint32_t counts = w[DVM_H_COUNTS];
  uint32_t n_tensors = counts & 0xff, n_in = (counts >> 8) & 0xff, n_opd = (counts >> 16) & 0xff;
  uint32_t geom = w[DVM_H_GEOM];
  int64_t n_tiles = w[DVM_H_N_TILES];
  int cores = dvm_get_num_cores();
  outf(o, "kernel vmain.vec  block_dim=%lld  body_tile=%lld  code_size=%u\n", (long long)n_tiles,
       (long long)((n_tiles + cores - 1) / cores), w[DVM_H_CODE_WORDS] * 4);
  outf(o, "  elems_per_thread=%u local_units=%u\n", w[DVM_H_LOCAL] >> 24, w[DVM_H_LOCAL2] >> 16);
  outf(o, "  rows=%llu cols=%u col_tile=%u col_blocks=%u threads_per_row=%u vec=%u local_regs=%u flags=%s%s%s\n",
       (unsigned long long)((uint64_t)w[DVM_H_ROWS_LO] | ((uint64_t)w[DVM_H_ROWS_HI] << 32)), w[DVM_H_COLS],
       w[DVM_H_COL_TILE], w[DVM_H_COL_BLOCKS], 1u << (geom & 0xff), (geom >> 8) & 0xff, (geom >> 16) & 0xff,
       ((geom >> 24) & DVM_F_ALIGNED) ? "A" : "-", ((geom >> 24) & DVM_F_OUTER_DIMS) ? "O" : "-",
       ((geom >> 24) & DVM_F_FLAT) ? "F" : "-");
  const uint32_t* ot = w + DVM_HDR_WORDS + 2 * n_tensors;
  for (uint32_t k = 0; k < n_opd; ++k) {
    const uint32_t* d = ot + k * DVM_OPD_WORDS;
    uint32_t info = d[0];
    outf(o, "  operand m%u: %s%u %s col_stride=%u strides=[%lld,%lld,%lld]%s\n", k,
         (info & 0xff) < n_in ? "in" : "out", (info & 0xff) < n_in ? (info & 0xff) : (info & 0xff) - n_in,
         ((info >> 8) & 0xff) == DVM_DT_BF16 ? "bf16" : ((info >> 8) & 0xff) == DVM_DT_U8 ? "u8" : ((info >> 8) & 0xff) == DVM_DT_I32 ? "i32" : "f32",
         ((info >> 16) & 0xff) ? d[DVM_OPD_COLSTRIDE] : 0u,
         (long long)d[2], (long long)d[4], (long long)d[6],
         (info >> 24) & 1 ? " primary" : (((info >> 26) & 3) == 1 ? " combine=sum" : ((info >> 26) & 3) == 2 ? " combine=max" : ((info >> 26) & 3) == 3 ? " combine=min" : ""));
  }
  const uint32_t* b = ot + n_opd * DVM_OPD_WORDS + ((geom >> 16) & 0xff);
  uint32_t body = w[DVM_H_CODE_WORDS], pc = 0;
  while (pc < body) {
    uint32_t w0 = b[pc], op = DVM_INSN_OP(w0), len = DVM_INSN_LEN(w0), a = DVM_INSN_A(w0), bb = DVM_INSN_B(w0);
    if (pc == w[DVM_H_LOAD_WORDS]) outf(o, "  ---- compute ----\n");
    outf(o, "  %04x: ", pc * 4);
    if (DVM_INSN_TAG(w0)) outf(o, "@p%u ", DVM_INSN_TAG(w0) - 1);  // runs in this phase only
    float imm = 0.f;
    if (len >= 2) memcpy(&imm, &b[pc + len - 1], 4);
    const char* dts = bb == DVM_DT_BF16 ? ".bf16" : "";
    if (op == DVM_OP_NOP) outf(o, "nop\n");
    else if (op == DVM_OP_PHASE) { if (a == 0xffu) outf(o, "phases    %u\n", bb); else outf(o, "end.below p%u\n", a); }
    else if (op == DVM_OP_LDG) outf(o, "load%s l%u, m%u\n", (a & 0x80) ? ".once" : "     ", a & 0x7f, bb);
    else if (op == DVM_OP_LDS) outf(o, "load.row  x%u, m%u\n", a, bb);
    else if (op == DVM_OP_LDA) outf(o, "copy      acc, l%u%s\n", a, dts);
    else if (op == DVM_OP_STA) outf(o, "copy      l%u, acc\n", a);
    else if (op == DVM_OP_LSS) outf(o, "copy      s%u, x%u\n", a, bb);
    else if (op == DVM_OP_STG) outf(o, "store     m%u, acc\n", bb);
    else if (op == DVM_OP_STS) outf(o, "store.row m%u, s%u\n", bb, a);
    else if (op == DVM_OP_BCS) outf(o, "broadcast acc, s%u\n", a);
    else if (op >= DVM_OP_BINI && op < DVM_OP_BINI + 8) outf(o, "%ss      acc, %.9g\n", kArith[op - DVM_OP_BINI], imm);
    else if (op >= DVM_OP_BIN && op < DVM_OP_BIN + 8) {
      if (a == DVM_REG_ACC) outf(o, "%-9s acc, acc, acc\n", kArith[op - DVM_OP_BIN]);
      else outf(o, "%-9s acc, acc, l%u%s\n", kArith[op - DVM_OP_BIN], a, dts);
    }
    else if (op >= DVM_OP_BINS && op < DVM_OP_BINS + 8) outf(o, "%-9s acc, acc, s%u\n", kArith[op - DVM_OP_BINS], a);
    else if (op >= DVM_OP_LD2 && op < DVM_OP_LD2 + 8)
      outf(o, "%-9s acc, l%u%s, l%u%s\n", kArith[op - DVM_OP_LD2], a, ((bb >> 6) & 1) ? ".bf16" : "", bb & 0x3f, (bb >> 7) ? ".bf16" : "");
    else if (op >= DVM_OP_CMP && op < DVM_OP_CMP + DVM_C_NCMP) {
      static const char* kCmp[DVM_C_NCMP] = {"cmp.gt", "cmp.ge", "cmp.lt", "cmp.le", "cmp.eq", "cmp.ne", "pow", "rpow"};
      if (a == DVM_REG_ACC) outf(o, "%-9s acc, acc, acc\n", kCmp[op - DVM_OP_CMP]);
      else outf(o, "%-9s acc, acc, l%u%s\n", kCmp[op - DVM_OP_CMP], a, dts);
    }
    else if (op == DVM_OP_SEL + 3) {
      float i1, i2;
      memcpy(&i1, &b[pc + 1], 4);
      memcpy(&i2, &b[pc + 2], 4);
      outf(o, "select    acc, acc ? %.9g : %.9g\n", i1, i2);
    }
    else if (op >= DVM_OP_SEL && op < DVM_OP_SEL + 3) {
      const char* s1 = ((bb >> 6) & 1) ? ".bf16" : "";
      const char* s2 = (bb >> 7) ? ".bf16" : "";
      if (op == DVM_OP_SEL) outf(o, "select    acc, acc ? l%u%s : l%u%s\n", a, s1, bb & 0x3f, s2);
      else if (op == DVM_OP_SEL + 1) outf(o, "select    acc, l%u%s ? l%u%s : acc\n", a, s1, bb & 0x3f, s2);
      else outf(o, "select    acc, l%u%s ? acc : l%u%s\n", a, s1, bb & 0x3f, s2);
    }
    else if (op >= DVM_OP_UN && op < DVM_OP_UN + DVM_U_NUN) outf(o, "%-9s acc, acc\n", kUn[op - DVM_OP_UN]);
    else if (op >= DVM_OP_ACT && op < DVM_OP_ACT + DVM_ACT_N) outf(o, "%-9s acc, acc\n", op == DVM_OP_ACT + DVM_ACT_GELU ? "gelu" : "silu");
    else if (op >= DVM_OP_RED && op < DVM_OP_RED + DVM_R_NRED) outf(o, "row%-6s s%u, acc\n", kRed[op - DVM_OP_RED], a);
    else if (op == DVM_OP_SOP) {
      uint32_t w1 = b[pc + 1], sub = w1 & 0xff, s1 = (w1 >> 8) & 0xff, s2 = (w1 >> 16) & 0xff;
      if (bb == DVM_SK_FMAU) {
        float m2, a2;
        memcpy(&m2, &b[pc + 2], 4); memcpy(&a2, &b[pc + 3], 4);
        outf(o, "s.fma%-5s s%u, s%u * %.9g + %.9g\n", sub == 0xff ? "" : kUn[sub], a, s1, m2, a2);
      }
      else if (bb == DVM_SK_BIN) outf(o, "s.%-7s s%u, s%u, s%u\n", kArith[sub], a, s1, s2);
      else if (bb == DVM_SK_BINI) outf(o, "s.%ss    s%u, s%u, %.9g\n", kArith[sub], a, s1, imm);
      else outf(o, "s.%-7s s%u, s%u\n", kUn[sub], a, s1);
    }
    pc += len;
  }
  return o.overflow ? DVM_ERR_BUFFER_TOO_SMALL : DVM_OK;
}

extern "C" int dvm_tensor_extents(const void* code, size_t code_size, int64_t* bytes_needed, int n_tensors) {
  if (!bytes_needed) return DVM_ERR_INVALID_ARG;
  int st = dvm_verify(code, code_size);
  if (st != DVM_OK) return st;
  const uint32_t* w = (const uint32_t*)code;
  const uint32_t counts = w[DVM_H_COUNTS];
  const uint32_t nt = counts & 0xff, n_opd = (counts >> 16) & 0xff;
  if ((uint32_t)n_tensors != nt) return DVM_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < nt; ++i) bytes_needed[i] = 0;
  if (w[DVM_H_N_TILES] == 0) return DVM_OK;
  auto need = [&](uint32_t slot, uint64_t last_element, uint32_t dt) {
    const int64_t b = (int64_t)((last_element + 1) << DVM_DT_LG_ES(dt));
    if (slot < nt && b > bytes_needed[slot]) bytes_needed[slot] = b;
  };
  if (w[DVM_H_KERNEL_TYPE] == DVM_KERNEL_MATMUL) {
    // A [M,K] and the B matrices [K,N] are dense bf16; epilogue operands are [M,N], [1,N] or [M,1] with a row stride
    const uint32_t* x = w + DVM_HDR_WORDS + 2 * nt;
    const uint64_t M = x[DVM_MM_M], N = x[DVM_MM_N], K = x[DVM_MM_K];
    need(x[DVM_MM_SLOTS] & 0xff, M * K - 1, DVM_DT_BF16);
    need((x[DVM_MM_SLOTS] >> 8) & 0xff, K * N - 1, DVM_DT_BF16);
    need((x[DVM_MM_SLOTS] >> 16) & 0xff, K * N - 1, DVM_DT_BF16);
    const uint32_t* ot = x + DVM_MM_WORDS;
    for (uint32_t o = 0; o < n_opd; ++o) {
      const uint32_t* d = ot + o * DVM_OPD_WORDS;
      const uint64_t rs = d[DVM_OPD_STRIDE0], cs = (d[DVM_OPD_INFO] >> 16) & 0xff;
      need(d[DVM_OPD_INFO] & 0xff, (M - 1) * rs + (N - 1) * cs, (d[DVM_OPD_INFO] >> 8) & 0xff);
    }
    return DVM_OK;
  }
  // vector programs: element (i2, i1, i0, col) of an operand lies at the sum of index x stride; the last row of a
  // flat program is shorter
  const uint32_t* ot = w + DVM_HDR_WORDS + 2 * nt;
  const uint64_t outer[3] = {w[DVM_H_OUTER0], w[DVM_H_OUTER1], w[DVM_H_OUTER2]};
  const uint64_t last_cols = w[DVM_H_LAST_ROW_COLS];
  for (uint32_t o = 0; o < n_opd; ++o) {
    const uint32_t* d = ot + o * DVM_OPD_WORDS;
    const uint32_t info = d[DVM_OPD_INFO];
    if ((info >> 26) & 3) {  // a combined result: dense, its element count in the descriptor
      need(info & 0xff, (uint64_t)d[DVM_OPD_FILL] - 1, DVM_DT_F32);
      continue;
    }
    uint64_t last = 0;
    for (int q = 0; q < 3; ++q) last += (outer[q] ? outer[q] - 1 : 0) * (uint64_t)d[DVM_OPD_STRIDE0 + 2 * q];
    if ((info >> 16) & 0xff) last += (last_cols - 1) * (uint64_t)d[DVM_OPD_COLSTRIDE];
    need(info & 0xff, last, (info >> 8) & 0xff);
  }
  return DVM_OK;
}

extern "C" int dvm_code_info(const void* code, size_t code_size, int* kernel_type, int64_t* n_tiles,
                             int* code_body_bytes, int* threads_per_row, int* vector_width, int* n_tile_regs) {
  int st = dvm_verify(code, code_size);
  if (st != DVM_OK) return st;
  const uint32_t* w = (const uint32_t*)code;
  if (kernel_type) *kernel_type = (int)w[DVM_H_KERNEL_TYPE];
  if (n_tiles) *n_tiles = w[DVM_H_N_TILES];
  if (code_body_bytes) *code_body_bytes = (int)w[DVM_H_CODE_WORDS] * 4;
  uint32_t geom = w[DVM_H_GEOM];
  if (threads_per_row) *threads_per_row = 1 << (geom & 0xff);
  if (vector_width) *vector_width = (geom >> 8) & 0xff;
  if (n_tile_regs) *n_tile_regs = (geom >> 16) & 0xff;
  return DVM_OK;
}

extern "C" const char* dvm_strerror(int status) {
  switch (status) {
    case DVM_OK: return "ok";
    case DVM_ERR_INVALID_ARG: return "invalid argument";
    case DVM_ERR_SHAPE_MISMATCH: return "shapes do not broadcast";
    case DVM_ERR_UNSUPPORTED: return "program not supported by the virtual machine";
    case DVM_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case DVM_ERR_BAD_CODE: return "bytecode failed verification";
    case DVM_ERR_CUDA: return "CUDA runtime error";
    case DVM_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case DVM_ERR_DEVICE_BAD_CODE: return "device met an undecodable instruction";
    case DVM_ERR_NOT_FINALIZED: return "program not finalized";
    case DVM_ERR_TOO_LARGE: return "program exceeds a library limit";
    default: return "unknown status";
  }
}
