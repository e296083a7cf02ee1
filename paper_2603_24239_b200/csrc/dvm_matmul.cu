// Matmul meta-kernel (Sec. 4.2 "matrix operations", Sec. 5.1 cube-vector fusion): the matmul
// instruction on the sm_100a tensor cores with the fused elementwise epilogue interpreted from bytecode.
//
//   out[M,N] = epilogue( A[M,K] x B_0[K,N] , A x B_1 , extra inputs )      bf16 operands, fp32 accumulate
//
// Host half: dvm_encode_matmul (shape check, output tiling, epilogue accumulator code), verifier, dump.
// Device half: one persistent CTA per SM, warp-specialised:
//   warp 0      one thread issues the TMA tile loads of a 4-stage shared-memory ring
//               (A: 128 x 64 K-major, B: 64 x 256 as four 64 x 64 boxes, 128-byte swizzle);
//   warp 1      one thread issues tcgen05.mma (M = 128, N = 256, K = 16 per instruction) into one of two
//               256-column accumulator stages of tensor memory and commits stage / tile completion to
//               mbarriers; with two B matrices the accumulator columns are [B_0 tile | B_1 tile], so the
//               gate and up products of one output tile sit side by side (the cube-vector constraint:
//               the epilogue needs matching tiles of both);
//   warps 2..5  the epilogue interpreter: every thread owns one output row of the tile, pulls
//               32-column chunks of the accumulators out of tensor memory (tcgen05.ld), runs the
//               epilogue code on them in registers and stores the narrowed result; it overlaps the
//               next tile's MMAs (the other accumulator stage).
// Two forms, chosen per launch (dvm_launch_matmul): single CTAs as above, or CTA pairs -- two CTAs of a cluster on
// a tile of 256 rows with tcgen05 cta_group::2, each loading its own A rows and half of the B tile (see
// dvm_mm_kernel).  In both, the tiles of a last, partial wave are shared along k among the CTAs (pairs) where
// that saves more than the exchange of the partial sums costs (see MMParams, mm_plan_split).
// Every wait on an mbarrier is bounded (time and iteration limit): when one runs out the CTA raises its
// abort flag, every role leaves its loop, copies and MMAs in flight are awaited (bounded again), tensor
// memory is released and the status word reports DVM_ERR_DEVICE_TIMEOUT.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "../../include/dvm.h"
#include "dvm_format.h"
#include "dvm_internal.h"
#include "dvm_launch.h"
#include "dvm_math.cuh"
#include "dvm_program.h"

// =================================================================================================
// Host: encode
// =================================================================================================
namespace {

constexpr int MM_MAX_BODY = 6 * DVM_MAX_NODES + 4 * DVM_MAX_TENSORS;

struct MmOperand {
  int slot, dtype, col_stride;
  int64_t row_stride;
};

struct MmEnc {
  const dvm_program* p;
  int16_t alias[DVM_MAX_NODES];
  int16_t uses[DVM_MAX_NODES];
  int16_t loc[DVM_MAX_NODES];  // register operand byte naming where the value lives, or -1
  int16_t tmp_val[DVM_MM_MAX_TMP];
  int n_tmp, nb;
  int16_t acc;
  uint32_t body[MM_MAX_BODY];
  int n_body;
  MmOperand opd[DVM_MAX_OPERANDS];
  int n_opd;
  bool stored[DVM_MAX_TENSORS];
  int8_t out_operand[DVM_MAX_TENSORS];
  const float* scalars;
  bool fail;
};

inline int mroot(const MmEnc& e, int v) {
  while (e.alias[v] >= 0) v = e.alias[v];
  return v;
}
inline void memit(MmEnc& e, uint32_t w) {
  if (e.n_body < MM_MAX_BODY) e.body[e.n_body++] = w;
  else e.fail = true;
}
inline uint32_t mf2u(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  return u;
}

void mm_spill_acc_if_live(MmEnc& e) {
  const int a = e.acc;
  if (a < 0 || e.uses[a] <= 0 || e.loc[a] >= 0) return;
  for (int k = 0; k < DVM_MM_MAX_TMP; ++k)
    if (e.tmp_val[k] < 0) {
      if (k + 1 > e.n_tmp) e.n_tmp = k + 1;
      memit(e, DVM_INSN(DVM_OP_STA, 1, e.nb + k, 0));
      e.tmp_val[k] = (int16_t)a;
      e.loc[a] = (int16_t)(e.nb + k);
      return;
    }
  e.fail = true;  // more live epilogue values than temporaries
}

void mm_ensure_acc(MmEnc& e, int v) {
  if (e.acc == v) return;
  mm_spill_acc_if_live(e);
  if (e.fail) return;
  if (e.loc[v] < 0) {
    e.fail = true;
    return;
  }
  memit(e, DVM_INSN(DVM_OP_LDA, 1, e.loc[v], 0));
  e.acc = (int16_t)v;
}

// One consumer of value v (held in a temporary) is done: free the temporary of a dead value.
void mm_release(MmEnc& e, int v) {
  if (e.uses[v] > 0) return;
  const int l = e.loc[v];
  if (l >= e.nb && l < e.nb + DVM_MM_MAX_TMP) {
    e.tmp_val[l - e.nb] = -1;
    e.loc[v] = -1;
  }
}

void mm_store_outputs_of(MmEnc& e, int v) {
  for (int o = 0; o < e.p->n_outputs; ++o) {
    if (e.stored[o] || mroot(e, e.p->outputs[o].value) != v) continue;
    mm_ensure_acc(e, v);
    if (e.fail) return;
    memit(e, DVM_INSN(DVM_OP_STG, 1, 0, e.out_operand[o]));
    e.stored[o] = true;
    e.uses[v]--;
  }
}

const uint8_t kMmBin[6] = {DVM_A_ADD, DVM_A_SUB, DVM_A_MUL, DVM_A_DIV, DVM_A_MIN, DVM_A_MAX};
inline uint8_t mm_reversed(uint8_t a) { return a == DVM_A_SUB ? DVM_A_RSUB : a == DVM_A_DIV ? DVM_A_RDIV : a; }

// Accumulator code of the elementwise epilogue (every value has the shape of the output tile).
bool mm_gen_epilogue(MmEnc& e) {
  const dvm_program* p = e.p;
  e.n_body = 0;
  e.n_tmp = 0;
  e.acc = -1;
  e.fail = false;
  for (int k = 0; k < DVM_MM_MAX_TMP; ++k) e.tmp_val[k] = -1;
  for (int o = 0; o < p->n_outputs; ++o) e.stored[o] = false;
  for (int i = 0; i < p->n_nodes; ++i) e.uses[i] = 0;
  for (int i = 0; i < p->n_nodes; ++i) {
    const Node& n = p->nodes[i];
    if (n.kind == NK_INPUT || n.kind == NK_MATMUL || e.alias[i] >= 0) continue;
    e.uses[mroot(e, n.x)]++;
    if (n.kind == NK_BINARY) e.uses[mroot(e, n.y)]++;
  }
  for (int o = 0; o < p->n_outputs; ++o) e.uses[mroot(e, p->outputs[o].value)]++;

  for (int i = 0; i < p->n_nodes && !e.fail; ++i) {
    const Node& n = p->nodes[i];
    if (n.kind == NK_INPUT || n.kind == NK_MATMUL || e.alias[i] >= 0) continue;
    if (e.uses[i] == 0) continue;  // dead value
    const int x = mroot(e, n.x);
    switch (n.kind) {
      case NK_UNARY:
      case NK_SCALAR:
      case NK_CAST: {
        mm_ensure_acc(e, x);
        if (e.fail) break;
        e.uses[x]--;
        mm_spill_acc_if_live(e);
        mm_release(e, x);
        if (n.kind == NK_UNARY) memit(e, DVM_INSN(DVM_OP_UN + n.op, 1, 0, 0));
        else if (n.kind == NK_CAST) memit(e, DVM_INSN(DVM_OP_UN + DVM_U_RND_BF16, 1, 0, 0));
        else {
          const float s = n.param >= 0 ? e.scalars[n.param] : n.imm;
          memit(e, DVM_INSN(DVM_OP_BINI + (n.op == DVM_ADDS ? DVM_A_ADD : DVM_A_MUL), 2, 0, 0));
          memit(e, mf2u(s));
        }
        e.acc = (int16_t)i;
        break;
      }
      case NK_BINARY: {
        const int y = mroot(e, n.y);
        uint8_t op = kMmBin[n.op];
        int other;  // the operand that is not in the accumulator
        if (e.acc == x) other = y;
        else if (e.acc == y) { other = x; op = mm_reversed(op); }
        else { mm_ensure_acc(e, x); other = y; }
        if (e.fail) break;
        const int held = e.acc;
        e.uses[x]--;
        e.uses[y]--;
        mm_spill_acc_if_live(e);
        if (e.fail) break;
        int operand;
        if (other == held) operand = DVM_REG_ACC;
        else if (e.loc[other] >= 0) operand = e.loc[other];
        else { e.fail = true; break; }
        memit(e, DVM_INSN(DVM_OP_BIN + op, 1, operand, 0));
        mm_release(e, x);
        if (y != x) mm_release(e, y);
        e.acc = (int16_t)i;
        break;
      }
      default:
        e.fail = true;
    }
    if (!e.fail) mm_store_outputs_of(e, i);
  }
  for (int o = 0; o < p->n_outputs && !e.fail; ++o)
    if (!e.stored[o]) mm_store_outputs_of(e, mroot(e, p->outputs[o].value));
  return !e.fail;
}

}  // namespace

int dvm_encode_matmul(const dvm_program* p, const dvm_shape* in_shapes, int n_in, const float* scalars,
                      int n_scalars, void* code, size_t code_capacity, size_t* code_size,
                      dvm_shape* out_shapes, int n_out) {
  (void)n_scalars;
  (void)n_out;
  MmEnc e;
  e.p = p;
  e.scalars = scalars;
  const int NN = p->n_nodes;

  // ---- the matmul instructions: one shared A [M,K], one or two B [K,N] ----
  int a_val = -1, b_val[2] = {-1, -1}, nb = 0;
  for (int i = 0; i < NN; ++i) {
    const Node& n = p->nodes[i];
    e.alias[i] = -1;
    e.loc[i] = -1;
    if (n.kind == NK_MATMUL) {
      if (nb >= 2) return DVM_ERR_UNSUPPORTED;
      a_val = n.x;
      b_val[nb] = n.y;
      e.loc[i] = (int16_t)nb;  // register nb: the accumulator of this matmul
      nb++;
    } else if (n.kind == NK_CAST && n.dtype == DVM_F32) {
      e.alias[i] = n.x;  // values are fp32 already
    } else if (n.kind == NK_CAST && n.dtype > DVM_BF16) {
      return DVM_ERR_UNSUPPORTED;  // integer types exist in vector programs only
    } else if (n.kind == NK_REDUCE) {
      return DVM_ERR_UNSUPPORTED;
    }
  }
  if (nb == 0) return DVM_ERR_INVALID_ARG;
  if (nb == 2 && b_val[0] == b_val[1]) return DVM_ERR_UNSUPPORTED;
  e.nb = nb;
  int slot_of[DVM_MAX_NODES];
  for (int i = 0; i < NN; ++i) slot_of[i] = -1;
  for (int i = 0; i < n_in; ++i) slot_of[p->inputs[i]] = i;
  const dvm_shape& sa = in_shapes[slot_of[a_val]];
  if (sa.rank != 2) return DVM_ERR_UNSUPPORTED;
  const int64_t M = sa.dims[0], K = sa.dims[1];
  int64_t N = -1;
  for (int j = 0; j < nb; ++j) {
    const dvm_shape& sb = in_shapes[slot_of[b_val[j]]];
    if (sb.rank != 2) return DVM_ERR_UNSUPPORTED;
    if (sb.dims[0] != K) return DVM_ERR_SHAPE_MISMATCH;
    if (N >= 0 && sb.dims[1] != N) return DVM_ERR_SHAPE_MISMATCH;
    N = sb.dims[1];
  }
  if (M < 0 || N < 0 || K < 0) return DVM_ERR_INVALID_ARG;
  // the tile loads want 16-byte row pitches; an empty inner dimension has no tensor-core form
  if (K <= 0 || (K % 8) != 0 || (N % 8) != 0) return DVM_ERR_UNSUPPORTED;
  if (M >= (1ll << 31) || N >= (1ll << 31) || K >= (1ll << 31)) return DVM_ERR_UNSUPPORTED;

  // ---- matmul operands feed only the matmul instructions; other inputs are epilogue operands ----
  e.n_opd = 0;
  for (int i = 0; i < NN; ++i) {
    const Node& n = p->nodes[i];
    if (n.kind == NK_INPUT || n.kind == NK_MATMUL) continue;
    const int xs[2] = {n.x, n.kind == NK_BINARY ? n.y : -1};
    for (int k = 0; k < 2; ++k)
      if (xs[k] >= 0 && (xs[k] == a_val || xs[k] == b_val[0] || xs[k] == b_val[1])) return DVM_ERR_UNSUPPORTED;
  }
  for (int o = 0; o < p->n_outputs; ++o) {
    const int v = p->outputs[o].value;
    if (v == a_val || v == b_val[0] || v == b_val[1]) return DVM_ERR_UNSUPPORTED;
  }
  for (int i = 0; i < n_in; ++i) {
    const int v = p->inputs[i];
    if (v == a_val || v == b_val[0] || v == b_val[1]) continue;
    const dvm_shape& s = in_shapes[i];
    if (s.rank != p->nodes[v].rank) return DVM_ERR_INVALID_ARG;
    if (s.rank > 2) return DVM_ERR_UNSUPPORTED;
    int64_t r = 1, c = 1;
    if (s.rank >= 1) c = s.dims[s.rank - 1];
    if (s.rank == 2) r = s.dims[0];
    if ((r != 1 && r != M) || (c != 1 && c != N)) return DVM_ERR_SHAPE_MISMATCH;
    if (e.n_opd >= DVM_MAX_OPERANDS) return DVM_ERR_TOO_LARGE;
    MmOperand& od = e.opd[e.n_opd];
    od.slot = i;
    od.dtype = p->nodes[v].dtype == DVM_BF16 ? DVM_DT_BF16 : DVM_DT_F32;
    od.col_stride = c == 1 ? 0 : 1;
    od.row_stride = r == 1 ? 0 : c;
    e.loc[v] = (int16_t)(0x80 | e.n_opd);
    e.n_opd++;
  }
  for (int o = 0; o < p->n_outputs; ++o) {
    if (e.n_opd >= DVM_MAX_OPERANDS) return DVM_ERR_TOO_LARGE;
    MmOperand& od = e.opd[e.n_opd];
    od.slot = n_in + o;
    if (p->outputs[o].dtype > DVM_BF16) return DVM_ERR_UNSUPPORTED;  // integer outputs exist in vector programs only
    od.dtype = p->outputs[o].dtype == DVM_BF16 ? DVM_DT_BF16 : DVM_DT_F32;
    od.col_stride = 1;
    od.row_stride = N;
    e.out_operand[o] = (int8_t)e.n_opd++;
    if (out_shapes) {
      out_shapes[o].rank = 2;
      out_shapes[o].dims[0] = M;
      out_shapes[o].dims[1] = N;
    }
  }

  if (!mm_gen_epilogue(e)) return DVM_ERR_UNSUPPORTED;

  // ---- output tiling: 128-row blocks x (128 | 256)-column blocks; one tile = one accumulator stage ----
  const int tile_n = nb == 2 ? 128 : 256;
  const int64_t mb = (M + DVM_MM_BLOCK_M - 1) / DVM_MM_BLOCK_M, nbk = (N + tile_n - 1) / tile_n;
  const int64_t kb = (K + DVM_MM_BLOCK_K - 1) / DVM_MM_BLOCK_K;
  if (mb * nbk >= (1ll << 31)) return DVM_ERR_UNSUPPORTED;

  const int nt = n_in + p->n_outputs;
  const size_t total = DVM_HDR_WORDS + 2 * (size_t)nt + DVM_MM_WORDS + (size_t)DVM_OPD_WORDS * e.n_opd + e.n_body;
  if (total > DVM_MM_MAX_WORDS) return DVM_ERR_TOO_LARGE;
  *code_size = total * 4;
  if (!code || code_capacity < total * 4) return DVM_ERR_BUFFER_TOO_SMALL;
  uint32_t* w = (uint32_t*)code;
  memset(w, 0, total * 4);
  w[DVM_H_MAGIC] = DVM_MAGIC;
  w[DVM_H_KERNEL_TYPE] = DVM_KERNEL_MATMUL;
  w[DVM_H_CODE_WORDS] = (uint32_t)e.n_body;
  w[DVM_H_N_TILES] = (uint32_t)(mb * nbk);
  w[DVM_H_TOTAL_WORDS] = (uint32_t)total;
  w[DVM_H_COUNTS] = (uint32_t)nt | ((uint32_t)n_in << 8) | ((uint32_t)e.n_opd << 16) | ((uint32_t)p->n_outputs << 24);
  w[DVM_H_COLS] = (uint32_t)N;
  w[DVM_H_ROWS_LO] = (uint32_t)M;
  w[DVM_H_PRIMARY] = 0xffffffffu;
  uint32_t* x = w + DVM_HDR_WORDS + 2 * nt;
  x[DVM_MM_M] = (uint32_t)M;
  x[DVM_MM_N] = (uint32_t)N;
  x[DVM_MM_K] = (uint32_t)K;
  x[DVM_MM_NB] = (uint32_t)nb;
  x[DVM_MM_TILE_N] = (uint32_t)tile_n;
  x[DVM_MM_SLOTS] = (uint32_t)slot_of[a_val] | ((uint32_t)slot_of[b_val[0]] << 8) |
                    ((uint32_t)slot_of[b_val[nb - 1]] << 16);
  x[DVM_MM_NTMP] = (uint32_t)e.n_tmp;
  x[DVM_MM_MBLOCKS] = (uint32_t)mb;
  x[DVM_MM_NBLOCKS] = (uint32_t)nbk;
  x[DVM_MM_KBLOCKS] = (uint32_t)kb;
  uint32_t* ot = x + DVM_MM_WORDS;
  for (int k = 0; k < e.n_opd; ++k) {
    uint32_t* d = ot + k * DVM_OPD_WORDS;
    d[DVM_OPD_INFO] = (uint32_t)e.opd[k].slot | ((uint32_t)e.opd[k].dtype << 8) | ((uint32_t)e.opd[k].col_stride << 16);
    d[DVM_OPD_STRIDE0] = (uint32_t)e.opd[k].row_stride;
    d[DVM_OPD_STRIDE0 + 1] = (uint32_t)((uint64_t)e.opd[k].row_stride >> 32);
  }
  memcpy(ot + e.n_opd * DVM_OPD_WORDS, e.body, (size_t)e.n_body * 4);
  return DVM_OK;
}

// =================================================================================================
// Host: verifier and readable dump
// =================================================================================================
namespace {
struct MmView {
  uint32_t nt, n_in, n_opd, n_out, nb, ntmp;
  const uint32_t *x, *ot, *body;
  uint32_t n_body;
};

bool mm_view(const uint32_t* w, size_t n_words, MmView* v) {
  if (n_words < DVM_HDR_WORDS || w[DVM_H_MAGIC] != DVM_MAGIC || w[DVM_H_KERNEL_TYPE] != DVM_KERNEL_MATMUL) return false;
  const uint32_t c = w[DVM_H_COUNTS];
  v->nt = c & 0xff; v->n_in = (c >> 8) & 0xff; v->n_opd = (c >> 16) & 0xff; v->n_out = c >> 24;
  if (v->nt > DVM_MAX_TENSORS || v->n_opd > DVM_MAX_OPERANDS || v->n_in + v->n_out != v->nt) return false;
  const size_t fixed = DVM_HDR_WORDS + 2 * (size_t)v->nt + DVM_MM_WORDS + (size_t)DVM_OPD_WORDS * v->n_opd;
  v->n_body = w[DVM_H_CODE_WORDS];
  if (w[DVM_H_TOTAL_WORDS] != n_words || fixed + v->n_body != n_words || n_words > DVM_MM_MAX_WORDS) return false;
  v->x = w + DVM_HDR_WORDS + 2 * v->nt;
  v->ot = v->x + DVM_MM_WORDS;
  v->body = v->ot + v->n_opd * DVM_OPD_WORDS;
  v->nb = v->x[DVM_MM_NB];
  v->ntmp = v->x[DVM_MM_NTMP];
  return true;
}

bool mm_reg_ok(const MmView& v, uint32_t r, bool allow_acc, bool temps_only) {
  if (temps_only) return r >= v.nb && r < v.nb + v.ntmp;
  if (r == DVM_REG_ACC) return allow_acc;
  if (r & 0x80) {
    const uint32_t k = r & 0x7f;
    return k < v.n_opd && (v.ot[k * DVM_OPD_WORDS] & 0xff) < v.n_in;
  }
  return r < v.nb + v.ntmp;
}
}  // namespace

int dvm_verify_matmul(const uint32_t* w, size_t n_words) {
  MmView v;
  if (!mm_view(w, n_words, &v)) return DVM_ERR_BAD_CODE;
  const uint32_t* x = v.x;
  const uint64_t M = x[DVM_MM_M], N = x[DVM_MM_N], K = x[DVM_MM_K];
  if (v.nb < 1 || v.nb > 2 || v.ntmp > DVM_MM_MAX_TMP) return DVM_ERR_BAD_CODE;
  if (x[DVM_MM_TILE_N] != (v.nb == 2 ? 128u : 256u)) return DVM_ERR_BAD_CODE;
  if (K == 0 || (K % 8) || (N % 8) || (M >> 31) || (N >> 31) || (K >> 31)) return DVM_ERR_BAD_CODE;
  const uint64_t mb = (M + DVM_MM_BLOCK_M - 1) / DVM_MM_BLOCK_M, nbk = (N + x[DVM_MM_TILE_N] - 1) / x[DVM_MM_TILE_N];
  if (x[DVM_MM_MBLOCKS] != mb || x[DVM_MM_NBLOCKS] != nbk || w[DVM_H_N_TILES] != mb * nbk) return DVM_ERR_BAD_CODE;
  if (x[DVM_MM_KBLOCKS] != (K + DVM_MM_BLOCK_K - 1) / DVM_MM_BLOCK_K) return DVM_ERR_BAD_CODE;
  if (w[DVM_H_COLS] != N || w[DVM_H_ROWS_LO] != M) return DVM_ERR_BAD_CODE;
  const uint32_t sl = x[DVM_MM_SLOTS];
  if ((sl & 0xff) >= v.n_in || ((sl >> 8) & 0xff) >= v.n_in || ((sl >> 16) & 0xff) >= v.n_in) return DVM_ERR_BAD_CODE;
  for (uint32_t k = 0; k < v.n_opd; ++k) {
    const uint32_t* d = v.ot + k * DVM_OPD_WORDS;
    const uint32_t info = d[DVM_OPD_INFO];
    if ((info & 0xff) >= v.nt || ((info >> 8) & 0xff) > DVM_DT_BF16 || ((info >> 16) & 0xff) > 1) return DVM_ERR_BAD_CODE;
    const uint64_t rs = d[DVM_OPD_STRIDE0] | ((uint64_t)d[DVM_OPD_STRIDE0 + 1] << 32);
    if (rs != 0 && rs != N && rs != 1) return DVM_ERR_BAD_CODE;
    if ((info & 0xff) >= v.n_in && (rs != N || ((info >> 16) & 0xff) != 1)) return DVM_ERR_BAD_CODE;  // outputs are dense
  }
  uint32_t pc = 0, stores = 0;
  while (pc < v.n_body) {
    const uint32_t iw = v.body[pc], op = DVM_INSN_OP(iw), len = DVM_INSN_LEN(iw), a = DVM_INSN_A(iw), b = DVM_INSN_B(iw);
    if (len == 0 || pc + len > v.n_body) return DVM_ERR_BAD_CODE;
    uint32_t want = 1;
    if (op == DVM_OP_LDA) { if (!mm_reg_ok(v, a, false, false)) return DVM_ERR_BAD_CODE; }
    else if (op == DVM_OP_STA) { if (!mm_reg_ok(v, a, false, true)) return DVM_ERR_BAD_CODE; }
    else if (op == DVM_OP_STG) {
      if (b >= v.n_opd || (v.ot[b * DVM_OPD_WORDS] & 0xff) < v.n_in) return DVM_ERR_BAD_CODE;
      stores++;
    }
    else if (op >= DVM_OP_BINI && op < DVM_OP_BINI + DVM_A_NBIN) want = 2;
    else if (op >= DVM_OP_BIN && op < DVM_OP_BIN + DVM_A_NBIN) { if (!mm_reg_ok(v, a, true, false)) return DVM_ERR_BAD_CODE; }
    else if (op >= DVM_OP_UN && op < DVM_OP_UN + DVM_U_RND_BF16 + 1) {}
    else return DVM_ERR_BAD_CODE;
    if (len != want) return DVM_ERR_BAD_CODE;
    pc += len;
  }
  if (stores == 0) return DVM_ERR_BAD_CODE;
  return DVM_OK;
}

namespace {
struct MmOut {
  char* buf;
  size_t cap, n;
};
void mm_printf(MmOut& o, const char* fmt, ...) {
  char tmp[256];
  va_list ap;
  va_start(ap, fmt);
  int k = vsnprintf(tmp, sizeof tmp, fmt, ap);
  va_end(ap);
  if (k < 0) return;
  for (int i = 0; i < k && i < (int)sizeof tmp - 1; ++i) {
    if (o.buf && o.n + 1 < o.cap) o.buf[o.n] = tmp[i];
    o.n++;
  }
}
const char* kMmArith[8] = {"add", "sub", "rsub", "mul", "div", "rdiv", "min", "max"};
const char* kMmUn[13] = {"exp", "sqrt", "rsqrt", "abs", "log", "erf", "sigmoid", "neg", "recip", "floor", "round", "tanh", "rnd_bf16"};
void mm_reg_name(const MmView& v, uint32_t r, char* out, size_t cap) {
  if (r == DVM_REG_ACC) snprintf(out, cap, "ACC");
  else if (r & 0x80) snprintf(out, cap, "G[%u]", r & 0x7f);
  else if (r < v.nb) snprintf(out, cap, "MM%u", r);
  else snprintf(out, cap, "T%u", r - v.nb);
}
}  // namespace

int dvm_disassemble_matmul(const uint32_t* w, size_t n_words, char* buf, size_t cap) {
  MmView v;
  if (!mm_view(w, n_words, &v)) return DVM_ERR_BAD_CODE;
  MmOut o = {buf, cap, 0};
  const uint32_t* x = v.x;
  mm_printf(o, "kernel matmul  code %u words  tiles %u (%u x %u, %u k-blocks)\n", v.n_body, w[DVM_H_N_TILES],
            x[DVM_MM_MBLOCKS], x[DVM_MM_NBLOCKS], x[DVM_MM_KBLOCKS]);
  mm_printf(o, "  M %u  N %u  K %u  B matrices %u  tile 128 x %u  temporaries %u\n", x[DVM_MM_M], x[DVM_MM_N],
            x[DVM_MM_K], v.nb, x[DVM_MM_TILE_N], v.ntmp);
  const uint32_t sl = x[DVM_MM_SLOTS];
  for (uint32_t j = 0; j < v.nb; ++j)
    mm_printf(o, "  MATMUL MM%u = slot%u x slot%u\n", j, sl & 0xff, (sl >> (8 + 8 * j)) & 0xff);
  for (uint32_t k = 0; k < v.n_opd; ++k) {
    const uint32_t* d = v.ot + k * DVM_OPD_WORDS;
    const uint32_t info = d[DVM_OPD_INFO];
    mm_printf(o, "  operand %u: slot%u %s row_stride %u col_stride %u\n", k, info & 0xff,
              ((info >> 8) & 0xff) == DVM_DT_BF16 ? "bf16" : "f32", d[DVM_OPD_STRIDE0], (info >> 16) & 0xff);
  }
  uint32_t pc = 0;
  char r[16];
  while (pc < v.n_body) {
    const uint32_t iw = v.body[pc], op = DVM_INSN_OP(iw), len = DVM_INSN_LEN(iw), a = DVM_INSN_A(iw), b = DVM_INSN_B(iw);
    if (len == 0 || pc + len > v.n_body) return DVM_ERR_BAD_CODE;
    mm_reg_name(v, a, r, sizeof r);
    if (op == DVM_OP_LDA) mm_printf(o, "  %3u: LDA   ACC = %s\n", pc, r);
    else if (op == DVM_OP_STA) mm_printf(o, "  %3u: STA   %s = ACC\n", pc, r);
    else if (op == DVM_OP_STG) mm_printf(o, "  %3u: STG   operand %u = ACC\n", pc, b);
    else if (op >= DVM_OP_BINI && op < DVM_OP_BINI + DVM_A_NBIN) {
      float f;
      memcpy(&f, &v.body[pc + 1], 4);
      mm_printf(o, "  %3u: BINI  ACC = ACC %s %g\n", pc, kMmArith[op & 7], f);
    } else if (op >= DVM_OP_BIN && op < DVM_OP_BIN + DVM_A_NBIN) mm_printf(o, "  %3u: BIN   ACC = ACC %s %s\n", pc, kMmArith[op & 7], r);
    else if (op >= DVM_OP_UN && op < DVM_OP_UN + DVM_U_RND_BF16 + 1) mm_printf(o, "  %3u: UN    ACC = %s(ACC)\n", pc, kMmUn[op - DVM_OP_UN]);
    else return DVM_ERR_BAD_CODE;
    pc += len;
  }
  if (buf && cap) buf[o.n < cap ? o.n : cap - 1] = 0;
  return o.n < cap ? DVM_OK : DVM_ERR_BUFFER_TOO_SMALL;
}

// =================================================================================================
// Device
// =================================================================================================
namespace dvm {
namespace mm {

constexpr int BLOCK_M = DVM_MM_BLOCK_M, BLOCK_K = DVM_MM_BLOCK_K, CHUNK = DVM_MM_CHUNK;
constexpr int ACC_COLS = 256;                       // accumulator columns of one tile (one UMMA N)
constexpr uint32_t STAGE_A = BLOCK_M * BLOCK_K * 2; // 16 KB: 128 rows of 128 bytes
constexpr uint32_t BOX_B = 64 * BLOCK_K * 2;        // 8 KB: 64 k-rows of 64 columns
constexpr uint32_t STAGE_BYTES = STAGE_A + 4 * BOX_B;  // 48 KB
constexpr int MAX_STAGES = 8;                       // barrier slots; 4 stages of 48 KB, or 6 to 7 of 32 KB for a CTA pair
constexpr uint32_t STAGE_PAIR = STAGE_A + 2 * BOX_B;  // 32 KB: this CTA's A rows and its half of the B tile
constexpr uint32_t STAGES_SINGLE = 4, STAGES_PAIR = 6;
constexpr uint32_t BAR_BYTES = 256;                  // barriers and flags behind the epilogue temporaries
constexpr uint32_t TMP_BYTES = 128 * CHUNK * 4;     // one epilogue temporary: 16 KB
constexpr int THREADS = 192;
constexpr uint32_t TMEM_COLS = 512;
constexpr unsigned long long WAIT_NS = 2000000000ull;   // limit of one wait: 2 s
constexpr unsigned long long DRAIN_NS = 200000000ull;   // limit of a wait for work in flight after an abort
constexpr uint32_t WAIT_SPINS = 1u << 27;

// Tail split (split_s >= 2): the tiles [split_first, split_first + split_r) -- the last, partial wave of the
// launch -- are shared along k.  Their k blocks form one line, tile a at [a * split_kbp, a * split_kbp + k_blocks);
// unit c (a CTA, or a CTA pair) takes the blocks [c * split_kb, (c + 1) * split_kb) of that line, i.e. a part of
// one tile, or the end of one tile and the start of the next.  Two layouts: a small last wave (at most half of
// the units) gives every tile s units of its own (split_kbp = s * split_kb: the parts are aligned to the tiles);
// a larger one is cut into equal ranges over all units (split_kbp = k_blocks: a tile has up to three parts).
// The unit holding a tile's first block owns it.  The other parts p = 1.. write their accumulators to `ws` (partial
// index a * (split_s - 1) + p - 1, laid out [column][row] fp32) and publish flags[4 a + p - 1] = epoch (on a CTA
// pair partial index and flag index are doubled, plus the CTA's rank: each CTA's 128 rows are a part of their
// own); the owner waits for them, adds them to its own accumulators in tensor memory in the order of p and runs
// the epilogue.  A unit works through its range in order, so it dumps (the end of a tile) before it waits (as the
// owner of the next): nobody waits for a unit that waits.  split_s is the largest number of parts of any tile.
struct MMParams {
  unsigned int* status;
  uint32_t pair_tiles, pair_mblocks;  // CTA pairs: tiles of 256 rows, blocks of 256 rows
  float* ws;
  uint32_t* flags;
  uint32_t epoch;
  uint32_t split_first, split_r, split_s, split_kb, split_kbp;
  uint32_t n_words;
  uint32_t n_stages;
  uint32_t words[DVM_MM_MAX_WORDS];
};
constexpr uint32_t MAX_SPLIT = 4;                    // parts of a tail tile at most
constexpr size_t PART_FLOATS = (size_t)BLOCK_M * ACC_COLS;  // one partial accumulator: 128 KB

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long gtimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: gives up after limit_ns (or WAIT_SPINS polls), raising the CTA's abort flag; with
// heed_abort it also gives up as soon as another role has raised the flag.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                            unsigned long long limit_ns, bool heed_abort) {
  const unsigned long long t0 = gtimer();
  for (uint32_t spin = 0; spin < WAIT_SPINS; ++spin) {
    if (mbar_try(bar, parity)) return true;
    if (heed_abort && *abort_flag) return false;
    if (gtimer() - t0 > limit_ns) break;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_try(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, WAIT_NS, true);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// mbarrier arrive once every tcgen05.mma issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// ---- the CTA-pair forms (tcgen05 cta_group::2: two CTAs of a cluster, one MMA over both their shared memories) ----
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// the shared::cluster address of `addr` (a shared-memory address of this CTA) in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t peer_addr(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// tile load of one CTA of a pair; the bytes are counted on `cluster_bar`, a barrier of the pair's first CTA
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on the barrier at this address in BOTH CTAs of the pair once the MMAs issued so far have completed
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}

// 32 consecutive accumulator columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[CHUNK]) {
  uint32_t r[CHUNK];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < CHUNK; ++i) v[i] = __uint_as_float(r[i]);
}

// the same 32 columns written back (the caller waits with tmem_st_wait before it reads them again)
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[CHUNK]) {
  uint32_t r[CHUNK];
#pragma unroll
  for (int i = 0; i < CHUNK; ++i) r[i] = __float_as_uint(v[i]);
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
      ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]),
        "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Bounded wait of a tile's owner for the n flags (`stride` words apart) of its other parts (each becomes `epoch` once that part's
// accumulators are in the workspace); like mbar_wait_slow it raises the CTA's abort flag when it gives up.
__device__ __noinline__ bool flags_wait(const uint32_t* f, uint32_t stride, uint32_t n, uint32_t epoch, volatile uint32_t* abort_flag) {
  const unsigned long long t0 = gtimer();
  uint32_t k = 0;
  for (uint32_t spin = 0; spin < WAIT_SPINS && k < n; ++spin) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(f + k * stride) : "memory");
    if (v == epoch) { ++k; continue; }
    if (*abort_flag) return false;
    if (gtimer() - t0 > WAIT_NS) break;
  }
  if (k == n) return true;
  *abort_flag = 1;
  return false;
}

// Shared-memory matrix descriptors (128-byte swizzle, sm_100 descriptor version 1).
// A tile, K-major: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t desc_k_major(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3fff) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// B tile, N-major: 64-column boxes 8192 bytes apart (leading offset), 8-deep k groups 1024 bytes apart.
__device__ __forceinline__ uint64_t desc_n_major(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3fff) | ((uint64_t)(BOX_B >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// kind::f16 instruction descriptor: fp32 accumulate, bf16 x bf16, A K-major, B N-major, M = 128, N = 256
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                           ((uint32_t)(ACC_COLS >> 3) << 17) | ((uint32_t)(BLOCK_M >> 4) << 24);
// the same over a CTA pair: M = 256
constexpr uint32_t IDESC_PAIR = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                                ((uint32_t)(ACC_COLS >> 3) << 17) | ((uint32_t)(2 * BLOCK_M >> 4) << 24);

__device__ __forceinline__ float mm_arith(int op, float a, float b) { return scalar_arith(op, a, b); }

// PAIR: two CTAs of a cluster work on one tile of 256 rows (128 each) with tcgen05 cta_group::2 -- each loads its
// own A rows and HALF of the B tile (the first CTA the accumulator columns 0..127, the second 128..255), the first
// CTA's MMA thread issues one instruction over both shared memories, both CTAs hold the accumulators of their own
// rows: a stage is 32 KB per CTA instead of 48, a third less traffic from L2 per flop.
template <bool PAIR>
__global__ void __launch_bounds__(THREADS, 1)
dvm_mm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
              const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ MMParams prm) {
#define MW(i) (prm.words[(i)])
  extern __shared__ uint8_t mm_smem_raw[];
  const uint32_t raw = smem_u32(mm_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;  // swizzled tiles want 1024-byte alignment
  uint8_t* const sm = mm_smem_raw + (base - raw);

  const uint32_t nt = MW(DVM_H_COUNTS) & 0xff, n_opd = (MW(DVM_H_COUNTS) >> 16) & 0xff;
  const uint32_t XO = DVM_HDR_WORDS + 2 * nt;       // matmul extension
  const uint32_t OT = XO + DVM_MM_WORDS;            // operand table
  const uint32_t CODE = OT + n_opd * DVM_OPD_WORDS; // epilogue code
  const uint32_t code_end = CODE + MW(DVM_H_CODE_WORDS);
  const int M = (int)MW(XO + DVM_MM_M), N = (int)MW(XO + DVM_MM_N);
  const int nb = (int)MW(XO + DVM_MM_NB), tile_n = (int)MW(XO + DVM_MM_TILE_N);
  const int ntmp = (int)MW(XO + DVM_MM_NTMP);
  const uint32_t m_blocks = MW(XO + DVM_MM_MBLOCKS), k_blocks = MW(XO + DVM_MM_KBLOCKS);
  const uint32_t n_tiles = MW(DVM_H_N_TILES);
  const uint32_t n_stages = prm.n_stages;

  constexpr uint32_t SB = PAIR ? STAGE_PAIR : STAGE_BYTES;          // bytes of one pipeline stage in this CTA
  const uint32_t tmp_base = n_stages * SB;                          // byte offsets from `base`
  const uint32_t bar_base = base + tmp_base + (uint32_t)ntmp * TMP_BYTES;
  // barriers: full[8] empty[8] tmem_full[2] tmem_empty[2] drain
  const uint32_t bar_full = bar_base, bar_empty = bar_base + 64, bar_tfull = bar_base + 128, bar_tempty = bar_base + 144,
                 bar_drain = bar_base + 160;
  uint32_t* const tmem_slot = (uint32_t*)(sm + tmp_base + (uint32_t)ntmp * TMP_BYTES + 176);
  volatile uint32_t* const abort_flag = tmem_slot + 1;
  const uint32_t rank = PAIR ? cluster_rank() : 0u;                 // 0: the pair's first CTA, which issues its MMAs

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < MAX_STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (uint32_t a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, PAIR ? 8 : 128);  // (a pair: one arrival per epilogue warp of both CTAs)
    }
    mbar_init(bar_drain, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // tensor memory: both accumulator stages
    if constexpr (PAIR) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync();  // the other CTA's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *(volatile uint32_t*)tmem_slot;

  // The i-th piece of work of this CTA: whole tiles blockIdx.x + i * gridDim.x below split_first, then (tail
  // split) one part of one tail tile.
  struct Work { uint32_t tile, kb0, kb1, part, parts, r; };
  // (a pair counts in clusters: its tiles, its grid)
  const uint32_t split_first = prm.split_s >= 2 ? prm.split_first : (PAIR ? prm.pair_tiles : n_tiles);
  const uint32_t unit = PAIR ? blockIdx.x >> 1 : blockIdx.x, n_units = PAIR ? gridDim.x >> 1 : gridDim.x;
  auto work_at = [&](uint32_t i, Work& w) -> bool {
    const uint32_t t = unit + i * n_units;
    w.part = 0; w.parts = 1; w.r = 0; w.kb0 = 0; w.kb1 = k_blocks;
    if (t < split_first) { w.tile = t; return true; }
    if (prm.split_s < 2) return false;
    // the q-th tile this unit's range of the tail's k blocks touches (split_first is a multiple of the units)
    const uint32_t q = (t - split_first) / n_units;
    const uint32_t W = prm.split_kb, kbp = prm.split_kbp;
    const uint32_t g0 = unit * W, gend = (prm.split_r - 1) * kbp + k_blocks;
    if (g0 >= gend) return false;
    const uint32_t g1 = min(g0 + W, gend);
    const uint32_t a = g0 / kbp + q;
    if (a >= prm.split_r) return false;
    const uint32_t s0 = max(g0, a * kbp), s1 = min(g1, a * kbp + k_blocks);
    if (s0 >= s1) return false;
    const uint32_t first_unit = (a * kbp) / W;  // the tile's owner
    w.r = a;
    w.tile = split_first + a;
    w.kb0 = s0 - a * kbp;
    w.kb1 = s1 - a * kbp;
    w.part = unit - first_unit;
    w.parts = (a * kbp + k_blocks - 1) / W - first_unit + 1;
    return true;
  };
  const bool split = prm.split_s >= 2;
  // first row and column of a tile for this CTA (a pair: blocks of 256 rows, this CTA's half of them)
  const uint32_t mbl = PAIR ? prm.pair_mblocks : m_blocks;
  auto tile_m0 = [&](uint32_t t) -> int { return (int)(t % mbl) * (PAIR ? 2 * BLOCK_M : BLOCK_M) + (int)rank * BLOCK_M; };
  auto tile_n0 = [&](uint32_t t) -> int { return (int)(t / mbl) * tile_n; };
  volatile uint32_t* const split_ok = tmem_slot + 2;

  uint32_t issued = 0, p_stage = 0, p_phase = 0;  // producer state, kept for the abort path
  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      bool ok = true;
      Work w;
      for (uint32_t i = 0; ok && work_at(i, w); ++i) {
        const uint32_t t = w.tile;
        const int m0 = tile_m0(t), n0 = tile_n0(t);
        for (uint32_t kb = w.kb0; kb < w.kb1; ++kb) {
          if (!mbar_wait(bar_empty + 8 * p_stage, p_phase ^ 1, abort_flag)) { ok = false; break; }
          const uint32_t full = bar_full + 8 * p_stage;
          const uint32_t sa = base + p_stage * SB;
          const int k0 = (int)kb * BLOCK_K;
          if constexpr (PAIR) {
            // both CTAs' bytes are counted on the first CTA's barrier, which alone expects them
            const uint32_t full0 = peer_addr(full, 0);
            if (rank == 0) mbar_expect_tx(full, 2 * SB);
            tma_load_2d_pair(sa, &tmA, full0, k0, m0);
            const CUtensorMap* mapb = (nb == 2 && rank == 1) ? &tmB1 : &tmB0;
            const int nh = n0 + (nb == 2 ? 0 : (int)rank * 128);
            tma_load_2d_pair(sa + STAGE_A, mapb, full0, nh, k0);
            tma_load_2d_pair(sa + STAGE_A + BOX_B, mapb, full0, nh + 64, k0);
            ++issued;
            if (++p_stage == n_stages) { p_stage = 0; p_phase ^= 1; }
            continue;
          }
          mbar_expect_tx(full, STAGE_BYTES);
          tma_load_2d(sa, &tmA, full, k0, m0);
          if (nb == 2) {
            tma_load_2d(sa + STAGE_A, &tmB0, full, n0, k0);
            tma_load_2d(sa + STAGE_A + BOX_B, &tmB0, full, n0 + 64, k0);
            tma_load_2d(sa + STAGE_A + 2 * BOX_B, &tmB1, full, n0, k0);
            tma_load_2d(sa + STAGE_A + 3 * BOX_B, &tmB1, full, n0 + 64, k0);
          } else {
#pragma unroll
            for (int b = 0; b < 4; ++b) tma_load_2d(sa + STAGE_A + b * BOX_B, &tmB0, full, n0 + 64 * b, k0);
          }
          ++issued;
          if (++p_stage == n_stages) { p_stage = 0; p_phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------- MMA issuer (a pair: the first CTA's) ----------------
    if (lane == 0 && rank == 0) {
      uint32_t stage = 0, phase = 0, it = 0;
      bool ok = true;
      Work w;
      for (; ok && work_at(it, w); ++it) {
        const uint32_t as = it & 1, aph = (it >> 1) & 1;
        if (!mbar_wait(bar_tempty + 8 * as, aph ^ 1, abort_flag)) break;  // the epilogue has drained this stage
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + as * ACC_COLS;
        for (uint32_t kb = w.kb0; kb < w.kb1; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = base + stage * SB;
          const uint64_t adesc = desc_k_major(sa), bdesc = desc_n_major(sa + STAGE_A);
#pragma unroll
          for (uint32_t j = 0; j < BLOCK_K / 16; ++j) {  // K = 16 per instruction: 32 bytes along A's rows, two k groups of B
            if constexpr (PAIR) umma_bf16_pair(d_tmem, adesc + 2 * j, bdesc + (uint64_t)(2048 >> 4) * j, IDESC_PAIR, ((kb - w.kb0) | j) != 0);
            else umma_bf16(d_tmem, adesc + 2 * j, bdesc + (uint64_t)(2048 >> 4) * j, IDESC, ((kb - w.kb0) | j) != 0);
          }
          // the stage is free once these MMAs have read it (a pair: in both CTAs)
          if constexpr (PAIR) umma_commit_pair(bar_empty + 8 * stage); else umma_commit(bar_empty + 8 * stage);
          if (++stage == n_stages) { stage = 0; phase ^= 1; }
        }
        if (ok) { if constexpr (PAIR) umma_commit_pair(bar_tfull + 8 * as); else umma_commit(bar_tfull + 8 * as); }
      }
    }
    __syncwarp();
  } else {
    // ---------------- epilogue interpreter ----------------
    const int q = warp & 3;                 // tensor-memory lane quadrant this warp may read
    const int erow = q * 32 + lane;         // row of the tile
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    float* const tmp_mine = (float*)(sm + tmp_base) + erow * 4;
    uint32_t it = 0;
    Work w;
    // the epilogue is done with accumulator stage `as` (a pair: told to the first CTA, whose MMA thread writes both
    // CTAs' accumulators, once per warp)
    auto release_acc = [&](uint32_t as) {
      if constexpr (PAIR) {
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(peer_addr(bar_tempty + 8 * as, 0));
      } else {
        mbar_arrive(bar_tempty + 8 * as);
      }
    };
    for (; work_at(it, w); ++it) {
      const uint32_t t = w.tile;
      const uint32_t as = it & 1, aph = (it >> 1) & 1;
      const bool got = mbar_wait(bar_tfull + 8 * as, aph, abort_flag);
      if (!__all_sync(0xffffffffu, got)) break;
      tc_fence_after();
      if (split && t >= split_first && w.parts > 1) {
        // ---- a tail tile computed in parts (see MMParams; a pair: each CTA's rows are a part of their own) ----
        constexpr uint32_t NR = PAIR ? 2 : 1;
        const uint32_t used_chunks = (uint32_t)(nb == 2 ? ACC_COLS : tile_n) / CHUNK;
        const uint32_t acc0 = lane_addr + as * ACC_COLS;
        if (w.part > 0) {  // this CTA's accumulators go to the workspace; the owner is told; nothing else to do here
          float* const dst0 = prm.ws + ((size_t)(w.r * (prm.split_s - 1) + (w.part - 1)) * NR + rank) * PART_FLOATS + erow;
          for (uint32_t c = 0; c < used_chunks; ++c) {
            float v[CHUNK];
            tmem_ld32(acc0 + c * CHUNK, v);
            float* dst = dst0 + (size_t)c * CHUNK * BLOCK_M;
#pragma unroll
            for (int k = 0; k < CHUNK; ++k) __stcg(dst + k * BLOCK_M, v[k]);  // (a warp's 32 rows of one column: one 128-byte line)
          }
          __threadfence();
          tc_fence_before();
          asm volatile("bar.sync 1, 128;" ::: "memory");
          if (threadIdx.x == 64) {
            uint32_t* f = prm.flags + (4 * w.r + (w.part - 1)) * NR + rank;
            asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(f), "r"(prm.epoch) : "memory");
          }
          release_acc(as);
          continue;
        }
        // the owner: every other part's accumulators, added in the order of the parts
        if (threadIdx.x == 64) {
          const bool ok = flags_wait(prm.flags + 4 * w.r * NR + rank, NR, w.parts - 1, prm.epoch, abort_flag);
          __threadfence();
          *split_ok = ok ? 1u : 0u;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (!*split_ok) break;
        for (uint32_t c = 0; c < used_chunks; ++c) {
          float v[CHUNK];
          tmem_ld32(acc0 + c * CHUNK, v);
          // (all loads of the chunk are issued before the first sum: the parts' lines come from L2 together)
          float x[MAX_SPLIT - 1][CHUNK];
#pragma unroll
          for (uint32_t p2 = 0; p2 < MAX_SPLIT - 1; ++p2) {
            const float* src = prm.ws + ((size_t)(w.r * (prm.split_s - 1) + p2) * NR + rank) * PART_FLOATS + (size_t)c * CHUNK * BLOCK_M + erow;
#pragma unroll
            for (int k = 0; k < CHUNK; ++k) x[p2][k] = p2 + 1 < w.parts ? __ldcg(src + k * BLOCK_M) : 0.0f;
          }
#pragma unroll
          for (uint32_t p2 = 0; p2 < MAX_SPLIT - 1; ++p2) {
#pragma unroll
            for (int k = 0; k < CHUNK; ++k) v[k] += x[p2][k];
          }
          tmem_st32(acc0 + c * CHUNK, v);
        }
        tmem_st_wait();
      }
      const int m0 = tile_m0(t), n0 = tile_n0(t);
      const int row = m0 + erow;
      const bool row_ok = row < M;
      const int n_chunks = tile_n / CHUNK;
      for (int c = 0; c < n_chunks; ++c) {
        const int col0 = n0 + c * CHUNK;
        if (col0 >= N) break;
        const uint32_t acc_addr = lane_addr + as * ACC_COLS + (uint32_t)(c * CHUNK);
        float acc[CHUNK];
#pragma unroll
        for (int i = 0; i < CHUNK; ++i) acc[i] = 0.0f;

        // operand `a` of LDA / BIN as CHUNK fp32 values
        auto fetch = [&](uint32_t a, float (&v)[CHUNK]) {
          if (a < (uint32_t)nb) {
            tmem_ld32(acc_addr + a * 128u, v);
          } else if (a < 0x80u) {
            const float4* src = (const float4*)(tmp_mine + (a - nb) * (TMP_BYTES / 4));
#pragma unroll
            for (int j = 0; j < CHUNK / 4; ++j) {
              const float4 f = src[j * 128];
              v[4 * j] = f.x; v[4 * j + 1] = f.y; v[4 * j + 2] = f.z; v[4 * j + 3] = f.w;
            }
          } else {
            const uint32_t od = OT + (a & 0x7fu) * DVM_OPD_WORDS;
            const uint32_t info = MW(od + DVM_OPD_INFO);
            const uint32_t slot = info & 0xff;
            const char* ptr = (const char*)(((unsigned long long)MW(DVM_HDR_WORDS + 2 * slot + 1) << 32) | MW(DVM_HDR_WORDS + 2 * slot));
            const long long rs = (long long)(((unsigned long long)MW(od + DVM_OPD_STRIDE0 + 1) << 32) | MW(od + DVM_OPD_STRIDE0));
            const int cs = (info >> 16) & 0xff;
            const bool bf = ((info >> 8) & 0xff) == DVM_DT_BF16;
            const long long off = (long long)row * rs + (long long)col0 * cs;
            const char* p0 = ptr + off * (bf ? 2 : 4);
            if (cs == 1 && col0 + CHUNK <= N && (((unsigned long long)p0) & 15) == 0) {
              // a whole chunk of a row-contiguous operand at an aligned address: 16-byte loads
              if (bf) {
#pragma unroll
                for (int g = 0; g < CHUNK / 8; ++g) {
                  uint4 q = make_uint4(0u, 0u, 0u, 0u);
                  if (row_ok) q = *(const uint4*)(p0 + 16 * g);
                  v[8 * g + 0] = __uint_as_float(q.x << 16); v[8 * g + 1] = __uint_as_float(q.x & 0xffff0000u);
                  v[8 * g + 2] = __uint_as_float(q.y << 16); v[8 * g + 3] = __uint_as_float(q.y & 0xffff0000u);
                  v[8 * g + 4] = __uint_as_float(q.z << 16); v[8 * g + 5] = __uint_as_float(q.z & 0xffff0000u);
                  v[8 * g + 6] = __uint_as_float(q.w << 16); v[8 * g + 7] = __uint_as_float(q.w & 0xffff0000u);
                }
              } else {
#pragma unroll
                for (int g = 0; g < CHUNK / 4; ++g) {
                  float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
                  if (row_ok) q = *(const float4*)(p0 + 16 * g);
                  v[4 * g] = q.x; v[4 * g + 1] = q.y; v[4 * g + 2] = q.z; v[4 * g + 3] = q.w;
                }
              }
            } else {
#pragma unroll
              for (int i = 0; i < CHUNK; ++i) {
                float x = 0.0f;
                if (row_ok && col0 + i < N) {
                  const long long e = off + (long long)i * cs;
                  x = bf ? __bfloat162float(((const __nv_bfloat16*)ptr)[e]) : ((const float*)ptr)[e];
                }
                v[i] = x;
              }
            }
          }
        };

        for (uint32_t pc = CODE; pc < code_end;) {
          const uint32_t iw = MW(pc);
          const uint32_t op = DVM_INSN_OP(iw), a = DVM_INSN_A(iw);
          if (op >= DVM_OP_BIN && op < DVM_OP_BIN + DVM_A_NBIN) {
            const int sub = op & 7;
            if (a == DVM_REG_ACC) {
#pragma unroll
              for (int i = 0; i < CHUNK; ++i) acc[i] = mm_arith(sub, acc[i], acc[i]);
            } else {
              float v[CHUNK];
              fetch(a, v);
              switch (sub) {
                case DVM_A_ADD:
#pragma unroll
                  for (int i = 0; i < CHUNK; ++i) acc[i] = acc[i] + v[i];
                  break;
                case DVM_A_MUL:
#pragma unroll
                  for (int i = 0; i < CHUNK; ++i) acc[i] = acc[i] * v[i];
                  break;
                default:
#pragma unroll
                  for (int i = 0; i < CHUNK; ++i) acc[i] = mm_arith(sub, acc[i], v[i]);
              }
            }
          } else if (op >= DVM_OP_UN && op < DVM_OP_UN + DVM_U_RND_BF16 + 1) {
            const int u = op - DVM_OP_UN;
            if (u == DVM_U_SIGMOID) {
#pragma unroll
              for (int i = 0; i < CHUNK; ++i) acc[i] = fast_rcp(1.0f + fast_exp(-acc[i]));
            } else {
#define DVM_MM_UN(U)                                                     \
  case U:                                                                \
    _Pragma("unroll") for (int i = 0; i < CHUNK; ++i) acc[i] = scalar_unary(U, acc[i]); \
    break;
              switch (u) {
                DVM_MM_UN(DVM_U_EXP) DVM_MM_UN(DVM_U_SQRT) DVM_MM_UN(DVM_U_RSQRT) DVM_MM_UN(DVM_U_ABS)
                DVM_MM_UN(DVM_U_LOG) DVM_MM_UN(DVM_U_NEG) DVM_MM_UN(DVM_U_RECIP)
                case DVM_U_ERF:  // on pairs: half as many polynomial chains as element by element
#pragma unroll
                  for (int i = 0; i < CHUNK; i += 2) {
                    const float2 r = packed_erf(make_float2(acc[i], acc[i + 1]));
                    acc[i] = r.x;
                    acc[i + 1] = r.y;
                  }
                  break;
                DVM_MM_UN(DVM_U_FLOOR) DVM_MM_UN(DVM_U_ROUND) DVM_MM_UN(DVM_U_TANH)
                default:
#pragma unroll
                  for (int i = 0; i < CHUNK; ++i) acc[i] = round_bf16(acc[i]);
              }
#undef DVM_MM_UN
            }
          } else if (op >= DVM_OP_BINI && op < DVM_OP_BINI + DVM_A_NBIN) {
            const float imm = __uint_as_float(MW(pc + 1));
            const int sub = op & 7;
#pragma unroll
            for (int i = 0; i < CHUNK; ++i) acc[i] = mm_arith(sub, acc[i], imm);
          } else if (op == DVM_OP_LDA) {
            fetch(a, acc);
          } else if (op == DVM_OP_STA) {
            float4* dst = (float4*)(tmp_mine + (a - nb) * (TMP_BYTES / 4));
#pragma unroll
            for (int j = 0; j < CHUNK / 4; ++j) dst[j * 128] = make_float4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
          } else if (op == DVM_OP_STG) {
            const uint32_t od = OT + DVM_INSN_B(iw) * DVM_OPD_WORDS;
            const uint32_t info = MW(od + DVM_OPD_INFO);
            const uint32_t slot = info & 0xff;
            char* ptr = (char*)(((unsigned long long)MW(DVM_HDR_WORDS + 2 * slot + 1) << 32) | MW(DVM_HDR_WORDS + 2 * slot));
            const bool bf = ((info >> 8) & 0xff) == DVM_DT_BF16;
            const bool vec = (((unsigned long long)ptr) & 15) == 0;  // N is a multiple of 8, col0 of 32
            if (row_ok) {
              const long long e0 = (long long)row * N + col0;
              if (bf) {
                __nv_bfloat16* o = (__nv_bfloat16*)ptr + e0;
                if (vec) {
#pragma unroll
                  for (int g = 0; g < CHUNK / 8; ++g) {
                    if (col0 + 8 * g < N) {
                      uint4 pk;
                      __nv_bfloat162 h;
                      h = __floats2bfloat162_rn(acc[8 * g], acc[8 * g + 1]);     pk.x = *(uint32_t*)&h;
                      h = __floats2bfloat162_rn(acc[8 * g + 2], acc[8 * g + 3]); pk.y = *(uint32_t*)&h;
                      h = __floats2bfloat162_rn(acc[8 * g + 4], acc[8 * g + 5]); pk.z = *(uint32_t*)&h;
                      h = __floats2bfloat162_rn(acc[8 * g + 6], acc[8 * g + 7]); pk.w = *(uint32_t*)&h;
                      *(uint4*)(o + 8 * g) = pk;
                    }
                  }
                } else {
#pragma unroll
                  for (int i = 0; i < CHUNK; ++i)
                    if (col0 + i < N) o[i] = __float2bfloat16_rn(acc[i]);
                }
              } else {
                float* o = (float*)ptr + e0;
                if (vec) {
#pragma unroll
                  for (int g = 0; g < CHUNK / 4; ++g)
                    if (col0 + 4 * g < N) *(float4*)(o + 4 * g) = make_float4(acc[4 * g], acc[4 * g + 1], acc[4 * g + 2], acc[4 * g + 3]);
                } else {
#pragma unroll
                  for (int i = 0; i < CHUNK; ++i)
                    if (col0 + i < N) o[i] = acc[i];
                }
              }
            }
          }
          pc += DVM_INSN_LEN(iw);
        }
      }
      // this accumulator stage may be overwritten by the tile after next
      tc_fence_before();
      release_acc(as);
    }
  }

  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (warp == 0 && lane == 0 && rank == 0) {
      // wait (bounded) for the tile loads still in flight: the latest fill of every stage (a pair: the first
      // CTA's barriers count both CTAs' bytes)
      uint32_t s = p_stage, ph = p_phase;
      const uint32_t n = issued < n_stages ? issued : n_stages;
      for (uint32_t i = 0; i < n; ++i) {
        if (s == 0) { s = n_stages - 1; ph ^= 1; } else --s;
        if (!mbar_try(bar_full + 8 * s, ph)) mbar_wait_slow(bar_full + 8 * s, ph, abort_flag, DRAIN_NS, false);
      }
    }
    if (warp == 1 && lane == 0 && rank == 0) {
      // wait (bounded) for every MMA issued so far
      if constexpr (PAIR) asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_drain) : "memory");
      else umma_commit(bar_drain);
      if (!mbar_try(bar_drain, 0)) mbar_wait_slow(bar_drain, 0, abort_flag, DRAIN_NS, false);
    }
    if (PAIR && rank == 1 && warp == 0) __nanosleep(50000);  // (this CTA's own last copies land meanwhile)
    if (threadIdx.x == 0) atomicMax(prm.status, (unsigned int)ST_TIMEOUT);
    __syncthreads();
  }
  // a pair leaves together: the first CTA's MMAs read the second one's shared memory and write its tensor memory
  if constexpr (PAIR) cluster_sync();
  if (warp == 1) {
    tc_fence_after();
    if constexpr (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
#undef MW
}

}  // namespace mm
}  // namespace dvm

// =================================================================================================
// Host: launch
// =================================================================================================
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

std::mutex g_mm_mu;
EncodeTiledFn g_encode_tiled = nullptr;
bool g_attr_set[64] = {};
int g_tail_split = 1;  // dvm_set_matmul_tail_split
int g_cta_pairs = 1;   // dvm_set_matmul_cta_pairs: 0 never, 1 where the cost estimate favours them, 2 wherever possible
int g_pair_clusters[64] = {};  // CTA pairs the device runs at a time (0: not asked yet, -1: none)

// Workspace of the tail split, one per (device, stream): launches of one stream run in order, so they may share
// it; launches of different streams may overlap, so they do not.  Allocated at the first launch that splits.
struct SplitSpace {
  int device;
  cudaStream_t stream;
  float* ws;
  uint32_t* flags;
  uint32_t epoch;
};
constexpr int MAX_SPLIT_SPACES = 16;
constexpr size_t SPLIT_WS_PARTS = 200;  // partial accumulators of 128 KB: a last wave of up to two thirds of 148 units with two exchanged parts per tile
constexpr size_t SPLIT_FLAG_WORDS = 4 * 160;
SplitSpace g_split[MAX_SPLIT_SPACES];
int g_n_split = 0;

// The workspace of (device, stream), or NULL (then the launch does not split): while the stream is being captured,
// or when every slot is taken.
SplitSpace* split_space(int device, cudaStream_t stream) {
  // A captured launch would be replayed with the epoch number it was captured with, which its flags then already
  // hold: launches into a capturing stream never split (nor would an allocation belong into a graph).
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) {
    cudaGetLastError();
    return nullptr;
  }
  std::lock_guard<std::mutex> lk(g_mm_mu);
  for (int i = 0; i < g_n_split; ++i)
    if (g_split[i].device == device && g_split[i].stream == stream) return &g_split[i];
  if (g_n_split == MAX_SPLIT_SPACES) return nullptr;
  SplitSpace sp = {device, stream, nullptr, nullptr, 0};
  if (cudaMalloc(&sp.ws, SPLIT_WS_PARTS * dvm::mm::PART_FLOATS * sizeof(float)) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  if (cudaMalloc(&sp.flags, SPLIT_FLAG_WORDS * 4) != cudaSuccess || cudaMemset(sp.flags, 0, SPLIT_FLAG_WORDS * 4) != cudaSuccess) {
    cudaGetLastError();
    cudaFree(sp.ws);
    if (sp.flags) cudaFree(sp.flags);
    return nullptr;
  }
  g_split[g_n_split] = sp;
  return &g_split[g_n_split++];
}

int mm_encode_fn(EncodeTiledFn* out) {
  std::lock_guard<std::mutex> lk(g_mm_mu);
  if (!g_encode_tiled) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
      dvm_note_cuda_error(e != cudaSuccess ? (int)e : (int)cudaErrorNotSupported);
      return DVM_ERR_CUDA;
    }
    g_encode_tiled = (EncodeTiledFn)fn;
  }
  *out = g_encode_tiled;
  return DVM_OK;
}

// A row-major bf16 matrix [rows, cols] as a 2-D tensor map with a (box_cols x box_rows) box, 128-byte swizzle.
int mm_make_map(EncodeTiledFn fn, CUtensorMap* map, void* ptr, uint64_t rows, uint64_t cols, uint32_t box_cols,
                uint32_t box_rows) {
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstride[1] = {cols * 2};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ptr, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    dvm_note_cuda_error((int)cudaErrorInvalidValue);
    return DVM_ERR_CUDA;
  }
  return DVM_OK;
}

}  // namespace

// Tail split of a launch of `tiles` tiles over `units` CTAs (or CTA pairs, nr = 2 CTAs each), see MMParams: the
// first tile of the last wave, its tiles, the most parts of a tile, the k blocks per unit and the tile pitch of
// the k line; false when the launch does not split.  A split saves the k blocks a unit no longer computes (0.47 us
// each) and costs the exchange: about 8 us, plus 0.2 us per 128-KB part that crosses L2 at the same moment
// (measured on both sweeps: two parts of 34 tiles on pairs cost 25 us, four parts of 2 tiles 10 us).
struct SplitPlan { uint32_t first, r, s, kb, kbp, units_used; double cost_blocks; };
constexpr double kUsPerKBlock = 0.47, kExchangeUs = 8.0, kUsPerPart = 0.2;
bool mm_plan_split(uint32_t tiles, uint32_t units, uint32_t kblocks, uint32_t nr, SplitPlan* sp) {
  const uint32_t tail = tiles % units;
  if (!g_tail_split || !tail || kblocks < 16) return false;
  sp->first = tiles - tail;
  sp->r = tail;
  double best = 0.0;  // microseconds gained
  if (2 * tail <= units) {  // every tile gets s units of its own, aligned parts: the best s
    uint32_t s_max = units / tail;
    if (s_max > dvm::mm::MAX_SPLIT) s_max = dvm::mm::MAX_SPLIT;
    for (uint32_t s_want = s_max; s_want >= 2; --s_want) {
      const uint32_t per = (kblocks + s_want - 1) / s_want;
      const uint32_t s_eff = (kblocks + per - 1) / per;
      if (s_eff < 2) continue;
      const double cost = kExchangeUs + kUsPerPart * tail * (s_eff - 1) * nr;
      const double gain = (kblocks - per) * kUsPerKBlock - cost;
      if (gain > best) {
        best = gain;
        sp->s = s_eff; sp->kb = per; sp->kbp = s_eff * per; sp->units_used = tail * s_eff;
        sp->cost_blocks = per + cost / kUsPerKBlock;
      }
    }
  } else {  // equal ranges of the tail's k line over all units: every unit dumps a part and owns a tile
    const uint32_t W = (uint32_t)(((uint64_t)tail * kblocks + units - 1) / units);
    uint32_t smax = 1, n_parts = 0;
    for (uint32_t a = 0; a < tail && W < kblocks; ++a) {
      const uint32_t parts = (a * kblocks + kblocks - 1) / W - (a * kblocks) / W + 1;
      if (parts > smax) smax = parts;
      n_parts += parts - 1;
    }
    const double cost = kExchangeUs + kUsPerPart * n_parts * nr;
    const double gain = W < kblocks ? (kblocks - W) * kUsPerKBlock - cost : 0.0;
    if (smax >= 2 && smax <= dvm::mm::MAX_SPLIT && gain > best) {
      best = gain;
      sp->s = smax; sp->kb = W; sp->kbp = kblocks; sp->units_used = (uint32_t)(((uint64_t)tail * kblocks + W - 1) / W);
      sp->cost_blocks = W + cost / kUsPerKBlock;
    }
  }
  if (best <= 0.0) return false;
  if ((size_t)tail * (sp->s - 1) * nr > SPLIT_WS_PARTS || (4 * (size_t)tail + 4) * nr > SPLIT_FLAG_WORDS) return false;
  return true;
}
// Estimated time of such a launch in tile times: the full waves, plus a last wave that costs a whole tile time, or
// with the tail split its longest share and the exchange.
double mm_waves(uint32_t tiles, uint32_t units, uint32_t kblocks, uint32_t nr) {
  double w = (double)(tiles / units);
  if (tiles % units) {
    SplitPlan sp;
    w += mm_plan_split(tiles, units, kblocks, nr, &sp) ? sp.cost_blocks / kblocks : 1.0;
  }
  return w;
}
// Whether a launch of mblocks x nblocks tiles (of 128 rows) should run on CTA pairs (tiles of 256 rows, over the
// clusters the device runs at a time): pairs run a tile 1.12 times faster (measured on the large launches of both
// sweeps: what a third less shared-memory traffic buys) but come in whole blocks of 256 rows and half as many units.
bool mm_prefers_pairs(uint32_t mblocks, uint32_t nblocks, uint32_t kblocks, uint32_t sms, uint32_t clusters) {
  if (g_cta_pairs >= 2) return true;
  const double single = mm_waves(mblocks * nblocks, sms, kblocks, 1);
  const double pair = mm_waves(((mblocks + 1) / 2) * nblocks, clusters, kblocks, 2) / 1.12;
  return pair < single;
}

int dvm_launch_matmul(const uint32_t* code, size_t n_words, void* const* tensors, int n_tensors, cudaStream_t stream) {
  MmView v;
  if (!mm_view(code, n_words, &v)) return DVM_ERR_BAD_CODE;
  if ((uint32_t)n_tensors != v.nt) return DVM_ERR_INVALID_ARG;
  if (code[DVM_H_N_TILES] == 0) return DVM_OK;  // an empty output launches nothing
  for (int i = 0; i < n_tensors; ++i)
    if (!tensors[i]) return DVM_ERR_INVALID_ARG;
  const uint32_t* x = v.x;
  const uint64_t M = x[DVM_MM_M], N = x[DVM_MM_N], K = x[DVM_MM_K];

  DvmDeviceInfo dev;
  int st = dvm_device_state(&dev);
  if (st != DVM_OK) return st;

  static thread_local dvm::mm::MMParams P;
  memcpy(P.words, code, n_words * 4);
  for (uint32_t i = 0; i < v.nt; ++i) {
    const unsigned long long a = (unsigned long long)(uintptr_t)tensors[i];
    P.words[DVM_HDR_WORDS + 2 * i] = (uint32_t)a;
    P.words[DVM_HDR_WORDS + 2 * i + 1] = (uint32_t)(a >> 32);
  }
  for (uint32_t k = 0; k < v.n_opd; ++k) {
    const uint32_t info = v.ot[k * DVM_OPD_WORDS];
    const uintptr_t es = ((info >> 8) & 0xff) == DVM_DT_BF16 ? 2 : 4;
    if ((uintptr_t)tensors[info & 0xff] % es) return DVM_ERR_INVALID_ARG;
  }
  const uint32_t sl = x[DVM_MM_SLOTS];
  void* pa = tensors[sl & 0xff];
  void* pb0 = tensors[(sl >> 8) & 0xff];
  void* pb1 = tensors[(sl >> 16) & 0xff];
  // the tile loads need 16-byte aligned matrices
  if (((uintptr_t)pa | (uintptr_t)pb0 | (uintptr_t)pb1) & 15) return DVM_ERR_INVALID_ARG;

  EncodeTiledFn fn;
  st = mm_encode_fn(&fn);
  if (st != DVM_OK) return st;
  CUtensorMap ma, mb0, mb1;
  if ((st = mm_make_map(fn, &ma, pa, M, K, DVM_MM_BLOCK_K, DVM_MM_BLOCK_M)) != DVM_OK) return st;
  if ((st = mm_make_map(fn, &mb0, pb0, K, N, 64, DVM_MM_BLOCK_K)) != DVM_OK) return st;
  if ((st = mm_make_map(fn, &mb1, pb1, K, N, 64, DVM_MM_BLOCK_K)) != DVM_OK) return st;

  // (both variants hold 192 KB of stages: 4 x 48 KB, or 6 x 32 KB per CTA of a pair)
  const size_t smem = 1024 + (size_t)dvm::mm::STAGES_SINGLE * dvm::mm::STAGE_BYTES + (size_t)v.ntmp * dvm::mm::TMP_BYTES +
                      dvm::mm::BAR_BYTES;
  static_assert(dvm::mm::STAGES_SINGLE * dvm::mm::STAGE_BYTES == dvm::mm::STAGES_PAIR * dvm::mm::STAGE_PAIR, "one shared-memory size");
  int devid = 0;
  DVM_CUDA(cudaGetDevice(&devid));
  if (devid < 0 || devid >= 64) return DVM_ERR_INVALID_ARG;
  int pair_clusters = 0;
  {
    std::lock_guard<std::mutex> lk(g_mm_mu);
    if (!g_attr_set[devid]) {
      DVM_CUDA(cudaFuncSetAttribute(dvm::mm::dvm_mm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448 - 1024));
      DVM_CUDA(cudaFuncSetAttribute(dvm::mm::dvm_mm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448 - 1024));
      g_attr_set[devid] = true;
    }
    if (g_pair_clusters[devid] == 0) {  // how many CTA pairs run at a time (with the largest shared-memory request)
      cudaLaunchConfig_t cfg = {};
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      cfg.gridDim = dim3(2 * (unsigned)dev.sm_count); cfg.blockDim = dim3(dvm::mm::THREADS);
      cfg.dynamicSmemBytes = 232448 - 1024; cfg.attrs = at; cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, dvm::mm::dvm_mm_kernel<true>, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
      g_pair_clusters[devid] = n > 0 ? n : -1;
    }
    pair_clusters = g_pair_clusters[devid] > 0 ? g_pair_clusters[devid] : 0;
  }
  P.status = dev.scratch;
  P.n_words = (uint32_t)n_words;
  P.n_stages = dvm::mm::STAGES_SINGLE;
  P.pair_tiles = P.pair_mblocks = 0;
  const uint32_t tiles = code[DVM_H_N_TILES];
  // CTA pairs (see dvm_mm_kernel): tiles of 256 rows
  const uint32_t mblocks = x[DVM_MM_MBLOCKS], nblocks = x[DVM_MM_NBLOCKS];
  if (g_cta_pairs && pair_clusters > 0 && mblocks >= 2 && mm_prefers_pairs(mblocks, nblocks, x[DVM_MM_KBLOCKS], (uint32_t)dev.sm_count, (uint32_t)pair_clusters)) {
    P.split_s = P.split_r = P.split_first = P.split_kb = P.split_kbp = 0;
    P.ws = nullptr; P.flags = nullptr; P.epoch = 0;
    // (an epilogue without temporaries leaves room for a seventh stage)
    P.n_stages = v.ntmp == 0 ? dvm::mm::STAGES_PAIR + 1 : dvm::mm::STAGES_PAIR;
    const size_t smem_pair = 1024 + (size_t)P.n_stages * dvm::mm::STAGE_PAIR + (size_t)v.ntmp * dvm::mm::TMP_BYTES + dvm::mm::BAR_BYTES;
    P.pair_mblocks = (mblocks + 1) / 2;
    P.pair_tiles = P.pair_mblocks * nblocks;
    uint32_t pairs = P.pair_tiles < (uint32_t)pair_clusters ? P.pair_tiles : (uint32_t)pair_clusters;
    SplitPlan plan;
    if (mm_plan_split(P.pair_tiles, (uint32_t)pair_clusters, x[DVM_MM_KBLOCKS], 2, &plan)) {
      if (SplitSpace* sp = split_space(devid, stream)) {
        P.split_first = plan.first; P.split_r = plan.r; P.split_s = plan.s; P.split_kb = plan.kb; P.split_kbp = plan.kbp;
        P.ws = sp->ws; P.flags = sp->flags;
        if (++sp->epoch == 0) sp->epoch = 1;
        P.epoch = sp->epoch;
        if (P.pair_tiles < (uint32_t)pair_clusters) pairs = plan.units_used;
      }
    }
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(dvm::mm::THREADS);
    cfg.dynamicSmemBytes = smem_pair; cfg.stream = stream; cfg.attrs = at; cfg.numAttrs = 1;
    DVM_CUDA(cudaLaunchKernelEx(&cfg, dvm::mm::dvm_mm_kernel<true>, ma, mb0, mb1, P));
    dvm_count_launch();
    return DVM_OK;
  }
  int grid = (int)(tiles < (uint32_t)dev.sm_count ? tiles : (uint32_t)dev.sm_count);
  // Tail split: the last wave of r <= sms / 2 tiles would leave most SMs idle for a whole tile time; instead
  // s = min(4, sms / r) CTAs take each of its tiles, a share of the k blocks each (see MMParams).
  P.split_s = P.split_r = P.split_first = P.split_kb = P.split_kbp = 0;
  P.ws = nullptr; P.flags = nullptr; P.epoch = 0;
  const uint32_t sms = (uint32_t)dev.sm_count;
  SplitPlan plan;
  if (mm_plan_split(tiles, sms, x[DVM_MM_KBLOCKS], 1, &plan)) {
    if (SplitSpace* sp = split_space(devid, stream)) {
      P.split_first = plan.first; P.split_r = plan.r; P.split_s = plan.s; P.split_kb = plan.kb; P.split_kbp = plan.kbp;
      P.ws = sp->ws; P.flags = sp->flags;
      if (++sp->epoch == 0) sp->epoch = 1;
      P.epoch = sp->epoch;
      if (tiles < sms) grid = (int)plan.units_used;
    }
  }
  dvm::mm::dvm_mm_kernel<false><<<grid, dvm::mm::THREADS, smem, stream>>>(ma, mb0, mb1, P);
  DVM_CUDA(cudaGetLastError());
  dvm_count_launch();
  return DVM_OK;
}

extern "C" void dvm_set_matmul_tail_split(int on) { g_tail_split = on; }

extern "C" int dvm_matmul_tail_plan(int64_t tiles, int units, int k_blocks, int ctas_per_unit, int32_t out[6]) {
  if (!out || tiles < 0 || tiles >= (1ll << 31) || units < 1 || k_blocks < 1 || ctas_per_unit < 1 || ctas_per_unit > 2)
    return DVM_ERR_INVALID_ARG;
  SplitPlan sp = {};
  if (!mm_plan_split((uint32_t)tiles, (uint32_t)units, (uint32_t)k_blocks, (uint32_t)ctas_per_unit, &sp)) return 0;
  out[0] = (int32_t)sp.first; out[1] = (int32_t)sp.r; out[2] = (int32_t)sp.s;
  out[3] = (int32_t)sp.kb; out[4] = (int32_t)sp.kbp; out[5] = (int32_t)sp.units_used;
  return 1;
}
extern "C" void dvm_set_matmul_cta_pairs(int mode) { g_cta_pairs = mode; }

// ---- self-test of the matmul kernel's bounded wait (see dvm_selftest_bounded_wait) ----
namespace dvm {
namespace mm {
__global__ void dvm_selftest_mm_wait_kernel(unsigned int* status) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ uint32_t abort_word;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    abort_word = 0;
    mbar_init(b, 2);  // two arrivals expected, one ever made: the phase never completes
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_arrive(b);
  }
  __syncthreads();
  const bool ok = mbar_wait(b, 0, &abort_word);
  __syncthreads();
  if (!ok && abort_word && threadIdx.x == 0) atomicMax(status, (unsigned int)ST_TIMEOUT);
}
}  // namespace mm
}  // namespace dvm

int dvm_selftest_mm_wait(unsigned int* status, cudaStream_t stream) {
  dvm::mm::dvm_selftest_mm_wait_kernel<<<1, 32, 0, stream>>>(status);
  DVM_CUDA(cudaGetLastError());
  dvm_count_launch();
  return DVM_OK;
}
