// Launch side of libdvm: sends a bytecode program to the device (as the kernel-parameter block)
// and starts the virtual machine on a persistent grid.
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <unordered_map>

#include "../../include/dvm.h"
#include "dvm_format.h"
#include "dvm_internal.h"
#include "dvm_launch.h"
#include "dvm_vm.cuh"
#include "dvm_vm_variants.h"
#include "dvm_link.h"

namespace {

constexpr int PW_SMALL = DVM_PW_SMALL;
constexpr int PW_LARGE = DVM_PW_LARGE;
constexpr int QUEUE_SLOTS = 504;
constexpr size_t SCRATCH_BYTES = (8 + 4 * QUEUE_SLOTS) * sizeof(unsigned int);
constexpr int MAX_DEVICES = 64;
constexpr size_t kMaxDynSmem = 227 * 1024 - 9 * 1024;  // dynamic shared memory a CTA may ask for (8.3 KB static part excluded)

struct DeviceState {
  bool ready = false;
  unsigned int* scratch = nullptr;  // [0] status word, [8 + 4*slot] work-queue counters (next tile, CTAs finished, tiles completed)
  int sm_count = 0;
  // resident CTAs per SM, per (kernel variant, bytes of dynamic shared memory / DVM_LOCAL_UNIT): occupancy depends
  // on exactly these two, so a one-slot and a two-slot launch of the same program never share an entry
  std::unordered_map<uint64_t, int> occ;
  unsigned queue_slot = 0;
};

DeviceState g_dev[MAX_DEVICES];
std::mutex g_mu;
thread_local int t_last_cuda_error = 0;
long long g_launches = 0;
thread_local const DvmVmVariant* t_last_variant = nullptr;  // dvm_last_launch_variant
int g_use_lean = 1;  // dvm_set_lean_kernel(0): every launch runs on the general interpreter (for comparisons)

}  // namespace

int dvm_device_state(DvmDeviceInfo* info) {
  int dev = 0;
  DVM_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEVICES) return DVM_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(g_mu);
  DeviceState& d = g_dev[dev];
  if (!d.ready) {
    DVM_CUDA(cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev));
    DVM_CUDA(cudaMalloc(&d.scratch, SCRATCH_BYTES));
    DVM_CUDA(cudaMemset(d.scratch, 0, SCRATCH_BYTES));
    d.ready = true;
  }
  info->scratch = d.scratch;
  info->sm_count = d.sm_count;
  info->queue_slot = d.queue_slot;
  d.queue_slot = (d.queue_slot + 1) % QUEUE_SLOTS;
  return DVM_OK;
}

// The groups of interpreter variants (dvm_vm_inst.cu, compiled once per group).
#define DVM_GROUPS(X) X(0) X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8) X(9) X(10) X(11) X(12) X(13) X(14) X(15) X(16) X(17) X(18) X(19) X(20) X(21) X(22) X(23) X(24) X(25) X(26) X(27) X(28) X(29) X(30) X(31) X(32) X(33) X(34) X(35) X(36) X(37) X(38) X(39) X(40) X(41) X(42) X(43) X(44) X(45) X(46) X(47) X(48) X(49) X(50)
#define DVM_DECL_GROUP(g) const DvmVmVariant* dvm_vm_group_##g(int* count);
DVM_GROUPS(DVM_DECL_GROUP)
#undef DVM_DECL_GROUP

const DvmVmVariant* dvm_vm_find_variant(int V, bool large, bool single, int ext, bool levels, int lean, bool heavy, int ctas) {
  typedef const DvmVmVariant* (*GroupFn)(int*);
#define DVM_GROUP_FN(g) &dvm_vm_group_##g,
  static const GroupFn groups[] = {DVM_GROUPS(DVM_GROUP_FN)};
#undef DVM_GROUP_FN
  for (GroupFn g : groups) {
    int n = 0;
    const DvmVmVariant* v = g(&n);
    for (int i = 0; i < n; ++i)
      if (v[i].V == V && v[i].large == (int)large && v[i].single == (int)single && v[i].ext == ext &&
          v[i].levels == (int)levels && v[i].lean == lean && (!lean || v[i].heavy == (int)heavy) && v[i].ctas == ctas)
        return &v[i];
  }
  return nullptr;
}

// Key of the occupancy cache: the variant and the dynamic shared memory in local-memory units.
uint64_t dvm_occupancy_key(const DvmVmVariant* v, size_t smem) {
  const uint64_t id = (uint64_t)v->V | ((uint64_t)v->large << 8) | ((uint64_t)v->single << 9) | ((uint64_t)v->ext << 10) |
                      ((uint64_t)v->levels << 12) | ((uint64_t)v->lean << 13) | ((uint64_t)v->heavy << 17) |  // (lean: four bits)
                      ((uint64_t)v->ctas << 18);
  return (id << 32) | (uint64_t)(smem / DVM_LOCAL_UNIT);
}

// Resident CTAs per SM of one interpreter variant for a launch with `smem` bytes of dynamic shared memory
// (cached per device).  The variants with level waits rely on the whole grid being resident: no CTA fits -> no launch.
// Two variants never share a cache key (a shared key would also skip the second kernel's shared-memory attribute).
static bool dvm_variant_keys_distinct() {
  typedef const DvmVmVariant* (*GroupFn)(int*);
#define DVM_GROUP_FN(g) &dvm_vm_group_##g,
  static const GroupFn groups[] = {DVM_GROUPS(DVM_GROUP_FN)};
#undef DVM_GROUP_FN
  std::unordered_map<uint64_t, const DvmVmVariant*> seen;
  for (GroupFn g : groups) {
    int n = 0;
    const DvmVmVariant* v = g(&n);
    for (int i = 0; i < n; ++i)
      if (!seen.emplace(dvm_occupancy_key(&v[i], 0), &v[i]).second) return false;
  }
  return true;
}

static int dvm_occupancy(const DvmVmVariant* v, size_t smem, int* out) {
  static const bool keys_ok = dvm_variant_keys_distinct();
  if (!keys_ok) return DVM_ERR_UNSUPPORTED;
  int dev = 0;
  DVM_CUDA(cudaGetDevice(&dev));
  std::lock_guard<std::mutex> lk(g_mu);
  DeviceState& d = g_dev[dev];
  const uint64_t key = dvm_occupancy_key(v, smem);
  auto it = d.occ.find(key);
  if (it == d.occ.end()) {
    int n = 0;
    DVM_CUDA(v->occupancy(smem, kMaxDynSmem, &n));
    if (n <= 0) {
      if (v->levels) return DVM_ERR_TOO_LARGE;
      n = 1;
    }
    it = d.occ.emplace(key, n).first;
  }
  *out = it->second;
  return DVM_OK;
}

void dvm_note_cuda_error(int e) { t_last_cuda_error = e; }
void dvm_count_launch() { __atomic_add_fetch(&g_launches, 1, __ATOMIC_RELAXED); }

extern "C" void dvm_set_lean_kernel(int on) { g_use_lean = on; }

extern "C" int dvm_last_launch_variant(int out[8]) {
  if (!out) return DVM_ERR_INVALID_ARG;
  const DvmVmVariant* v = t_last_variant;
  if (!v) return DVM_ERR_INVALID_ARG;
  out[0] = v->V; out[1] = v->large; out[2] = v->single; out[3] = v->ext;
  out[4] = v->levels; out[5] = v->lean; out[6] = v->heavy; out[7] = v->ctas;
  return DVM_OK;
}
static int g_stacked_one_slot = 0;
extern "C" void dvm_set_stacked_one_slot(int on) { g_stacked_one_slot = on != 0; }
extern "C" int dvm_last_cuda_error(void) { return t_last_cuda_error; }
extern "C" int64_t dvm_launch_count(void) { return (int64_t)__atomic_load_n(&g_launches, __ATOMIC_RELAXED); }

namespace {

// Copies one verified vector program into `dst` and patches in what only the launch knows: the tensor
// addresses, each input register's address phase (address modulo 16), and -- when the program assumed
// 16-byte aligned rows but the primary operand's base pointer is not -- the switch to address-derived shifts.
int place_program(uint32_t* dst, const uint32_t* code, void* const* tensors, int n_tensors) {
  const uint32_t total = code[DVM_H_TOTAL_WORDS];
  memcpy(dst, code, (size_t)total * 4);
  const uint32_t counts = code[DVM_H_COUNTS];
  const uint32_t nt = counts & 0xff, n_opd = (counts >> 16) & 0xff;
  if ((uint32_t)n_tensors != nt) return DVM_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < nt; ++i) {
    if (!tensors[i]) return DVM_ERR_INVALID_ARG;
    unsigned long long a = (unsigned long long)(uintptr_t)tensors[i];
    dst[DVM_HDR_WORDS + 2 * i] = (uint32_t)a;
    dst[DVM_HDR_WORDS + 2 * i + 1] = (uint32_t)(a >> 32);
  }
  const uint32_t* ot = code + DVM_HDR_WORDS + 2 * nt;
  for (uint32_t o = 0; o < n_opd; ++o) {
    uint32_t info = ot[o * DVM_OPD_WORDS];
    uintptr_t a = (uintptr_t)tensors[info & 0xff];
    uintptr_t es = (uintptr_t)1 << DVM_DT_LG_ES((info >> 8) & 0xff);
    if (a % es) return DVM_ERR_INVALID_ARG;
  }
  // every input register learns its tensor's address modulo 16 (the images keep that phase)
  {
    const uint32_t n_inr = code[DVM_H_LOCAL] & 0xff;
    uint32_t* lt = dst + DVM_HDR_WORDS + 2 * nt + n_opd * DVM_OPD_WORDS;
    for (uint32_t k = 0; k < n_inr; ++k) {
      const uint32_t info = ot[(lt[k] >> 24) * DVM_OPD_WORDS];
      lt[k] = (lt[k] & ~(0xfu << 20)) | (((uint32_t)(uintptr_t)tensors[info & 0xff] & 15u) << 20);
    }
  }
  // A program encoded for aligned rows relies on a 16-byte aligned primary tensor; on any other base address
  // the interpreter derives the row shift from the actual address instead (the rows' last columns then
  // wrap around into the head slots when a row fills its whole capacity).
  const uint32_t geom = code[DVM_H_GEOM];
  const uint32_t flags = geom >> 24;
  if ((flags & DVM_F_ALIGNED) && code[DVM_H_PRIMARY] != 0xffffffffu) {
    const uint32_t info = ot[code[DVM_H_PRIMARY] * DVM_OPD_WORDS];
    if (((uintptr_t)tensors[info & 0xff]) & 15) dst[DVM_H_GEOM] = geom & ~((uint32_t)DVM_F_ALIGNED << 24);
  }
  return DVM_OK;
}


// ---- the linker of the lean interpreter (see dvm_link.h) ----
// Turns the placed copy of one verified vector program at dst (word index `at` of the parameter block) into its
// linked form: header, tables and load section stay, the compute section is replaced by records (which start at
// a word index = 0 mod 4 of the block: 16-byte aligned in the kernel's parameter space).  `src` is the encoded
// program, `tensors` its device pointers, `max_words` the room at dst.  Returns the words the linked program
// takes, or 0 when it cannot be linked (no room, or an instruction only the general interpreter has).
uint32_t dvm_link_program(uint32_t* dst, uint32_t at, uint32_t max_words, const uint32_t* src, void* const* tensors) {
  const uint32_t counts = src[DVM_H_COUNTS], geom = src[DVM_H_GEOM];
  const uint32_t nt = counts & 0xff, n_opd = (counts >> 16) & 0xff, nreg = (geom >> 16) & 0xff;
  const uint32_t tables = DVM_HDR_WORDS + 2 * nt + n_opd * DVM_OPD_WORDS + nreg;
  const uint32_t load_words = src[DVM_H_LOAD_WORDS], code_words = src[DVM_H_CODE_WORDS];
  const uint32_t head = tables + load_words;  // header, tables and load section: copied as they are
  if (n_opd > 63) return 0;
  const uint32_t* ot = src + DVM_HDR_WORDS + 2 * nt;
  const uint32_t* lt = dst + DVM_HDR_WORDS + 2 * nt + n_opd * DVM_OPD_WORDS;  // (the placed table: address phases patched in)
  const uint32_t* body = src + tables;
  const uint32_t scalar_unit = src[DVM_H_LOCAL2] & 0xffffu;
  struct Rec { uint32_t w[4]; };
  Rec rec[8 * DVM_MAX_NODES + 72];
  uint32_t n = 0;
  auto push = [&](uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3) {
    rec[n].w[0] = w0; rec[n].w[1] = w1; rec[n].w[2] = w2; rec[n].w[3] = w3;
    ++n;
  };
  auto f2u = [](float f) { uint32_t u; memcpy(&u, &f, 4); return u; };
  auto u2f = [](uint32_t u) { float f; memcpy(&f, &u, 4); return f; };
  // every output of the program is bf16: the one-piece exponential is accurate enough
  bool fast = true;
  for (uint32_t o = n_opd - (counts >> 24); o < n_opd; ++o)
    if (((ot[o * DVM_OPD_WORDS + DVM_OPD_INFO] >> 8) & 0xff) != DVM_DT_BF16) fast = false;
  // operand word of local register k holding elements of type dt
  auto opw = [&](uint32_t k, uint32_t dt, int* kind) -> uint32_t {
    const uint32_t lw = lt[k];
    const uint32_t mode = (lw >> 16) & 0xf;
    *kind = mode == DVM_LM_PRIVATE ? 2 : (dt == DVM_DT_BF16 ? 0 : 1);
    return DVM_LK_OPW((lw & 0xffffu) * DVM_LOCAL_UNIT, mode, dt == DVM_DT_BF16 ? 0 : 1, (lw >> 20) & 0xfu, lw >> 24);
  };
  const float one = 1.0f, neg_one = -1.0f, neg_zero = -0.0f;
  // handlers by kind of operand (0 bf16 image, 1 fp32 image, 2 private temporary)
  static const uint32_t kLda[3] = {DVM_LK_LDA_BF16, DVM_LK_LDA_F32, DVM_LK_LDA_PRIV};
  static const uint32_t kBin[3] = {DVM_LK_BIN_BF16, DVM_LK_BIN_F32, DVM_LK_BIN_PRIV};
  for (uint32_t pc = load_words; pc < code_words;) {
    if (n + 4 > sizeof rec / sizeof rec[0]) return 0;
    const uint32_t w0 = body[pc], op = DVM_INSN_OP(w0), len = DVM_INSN_LEN(w0) ? DVM_INSN_LEN(w0) : 1;
    const uint32_t ia = DVM_INSN_A(w0), ib = DVM_INSN_B(w0);
    const uint32_t cls = op >> 3;
    const uint32_t tag = DVM_INSN_TAG(w0);  // phased programs: the phase a run-once instruction belongs to
    int kind = 0;
    if (op == DVM_OP_PHASE) {
      if (ia != 0xffu) push(DVM_LK_W0(DVM_LK_PHASE, 0, ia, 0), 0, 0, 0);
    } else if (op == DVM_OP_LDA) {
      const uint32_t ow = opw(ia, ib, &kind);
      push(DVM_LK_W0(kLda[kind], 0, 0, 0), ow, 0, 0);
    } else if (cls == (DVM_OP_LD2 >> 3)) {
      const uint32_t ox = opw(ia, (ib >> 6) & 1, &kind);
      push(DVM_LK_W0(kLda[kind], 0, 0, 0), ox, 0, 0);
      const uint32_t oy = opw(ib & 0x3f, (ib >> 7) & 1, &kind);
      push(DVM_LK_W0(kBin[kind], op & 7, 0, 0), oy, 0, 0);
    } else if (cls == (DVM_OP_BIN >> 3)) {
      if (ia == DVM_REG_ACC) {
        push(DVM_LK_W0(DVM_LK_BIN_ACC, op & 7, 0, 0), 0, 0, 0);
      } else {
        const uint32_t oy = opw(ia, ib, &kind);
        push(DVM_LK_W0(kBin[kind], op & 7, 0, 0), oy, 0, 0);
      }
    } else if (cls == (DVM_OP_BINI >> 3)) {
      const float y = u2f(body[pc + 1]);
      switch (op & 7) {  // ACC * m + c (a product plus -0 is the product, sign of zero included)
        case DVM_A_ADD: push(DVM_LK_W0(DVM_LK_FMA, 0, 0, 0), f2u(one), f2u(y), 0); break;
        case DVM_A_SUB: push(DVM_LK_W0(DVM_LK_FMA, 0, 0, 0), f2u(one), f2u(-y), 0); break;
        case DVM_A_RSUB: push(DVM_LK_W0(DVM_LK_FMA, 0, 0, 0), f2u(neg_one), f2u(y), 0); break;
        case DVM_A_MUL: push(DVM_LK_W0(DVM_LK_FMA, 0, 0, 0), f2u(y), f2u(neg_zero), 0); break;
        case DVM_A_DIV: push(DVM_LK_W0(DVM_LK_FMA, 4, 0, 0), f2u(y), f2u(neg_zero), 0); break;  // the device's reciprocal, as for S[a]
        default: push(DVM_LK_W0(DVM_LK_BINI, op & 7, 0, 0), body[pc + 1], 0, 0); break;
      }
    } else if (cls == (DVM_OP_BINS >> 3)) {
      // ACC = ACC - S[a] ; exp  ->  EXPS
      const uint32_t nx = pc + len < code_words ? body[pc + len] : 0;
      if ((op & 7) == DVM_A_SUB && pc + len < code_words && DVM_INSN_OP(nx) == DVM_OP_UN + DVM_U_EXP) {
        push(DVM_LK_W0(DVM_LK_EXPS, fast ? 1 : 0, ia, 0), 0, 0, 0);
        pc += 1;  // (the unary has one word)
      } else {
        switch (op & 7) {
          case DVM_A_ADD: push(DVM_LK_W0(DVM_LK_FMA, 2, 0, ia), f2u(one), 0, 0); break;
          case DVM_A_SUB: push(DVM_LK_W0(DVM_LK_FMA, 2 | 8, 0, ia), f2u(one), 0, 0); break;
          case DVM_A_RSUB: push(DVM_LK_W0(DVM_LK_FMA, 2, 0, ia), f2u(neg_one), 0, 0); break;
          case DVM_A_MUL: push(DVM_LK_W0(DVM_LK_FMA, 1, ia, 0), 0, f2u(neg_zero), 0); break;
          case DVM_A_DIV: push(DVM_LK_W0(DVM_LK_FMA, 1 | 4, ia, 0), 0, f2u(neg_zero), 0); break;
          default: push(DVM_LK_W0(DVM_LK_BINS, op & 7, ia, 0), 0, 0, 0); break;
        }
      }
    } else if (op >= DVM_OP_UN && op < DVM_OP_UN + DVM_U_NUN) {
      const uint32_t u = op - DVM_OP_UN;
      if (u == DVM_U_ISFINITE) return 0;
      push(DVM_LK_W0(DVM_LK_UN, u | ((fast && (u == DVM_U_EXP || u == DVM_U_SIGMOID)) ? 0x80u : 0u), 0, 0), 0, 0, 0);
    } else if (op >= DVM_OP_ACT && op < DVM_OP_ACT + DVM_ACT_N) {
      push(DVM_LK_W0(DVM_LK_ACT, op - DVM_OP_ACT, 0, 0), 0, 0, 0);
    } else if (cls == (DVM_OP_RED >> 3)) {
      // RED ; SOP fma(-unary) that reads the result and overwrites it  ->  one reduction with a post-operation
      const uint32_t nx = pc + len < code_words ? body[pc + len] : 0;
      bool fused = false;
      if (pc + len < code_words && DVM_INSN_OP(nx) == DVM_OP_SOP && DVM_INSN_B(nx) == DVM_SK_FMAU) {
        const uint32_t w1 = body[pc + len + 1];
        if (((w1 >> 8) & 0xff) == ia && DVM_INSN_A(nx) == ia && DVM_INSN_TAG(nx) == tag) {
          push(DVM_LK_W0(DVM_LK_RED, op & 7, ia, 1 | (tag << 4)), w1 & 0xff, body[pc + len + 2], body[pc + len + 3]);
          pc += DVM_INSN_LEN(nx);
          fused = true;
        }
      }
      if (!fused) push(DVM_LK_W0(DVM_LK_RED, op & 7, ia, tag << 4), 0, 0, 0);
    } else if (op == DVM_OP_STG) {
      const uint32_t info = ot[ib * DVM_OPD_WORDS + DVM_OPD_INFO];
      if (!((info >> 25) & 1u) || ((info >> 26) & 3u)) return 0;  // a stored view / a combined result: general interpreter
      const unsigned long long a = (unsigned long long)(uintptr_t)tensors[info & 0xff];
      const uint32_t sdt = (info >> 8) & 0xff;   // sub: 0 fp32 / bf16 as they are, 1: converted to i32, 2: to u8
      push(DVM_LK_W0(sdt > DVM_DT_BF16 ? DVM_LK_STGI : DVM_LK_STG, sdt == DVM_DT_I32 ? 1 : sdt == DVM_DT_U8 ? 2 : 0, DVM_DT_LG_ES(sdt), tag), (uint32_t)a, (uint32_t)(a >> 32), 0);
    } else if (op == DVM_OP_STA) {
      push(DVM_LK_W0(DVM_LK_STA, 0, 0, 0), (lt[ia] & 0xffffu) * DVM_LOCAL_UNIT, 0, 0);
    } else if (op == DVM_OP_LSS) {
      push(DVM_LK_W0(DVM_LK_LSS, 0, ia, 0), scalar_unit * DVM_LOCAL_UNIT + (ib >> 2) * (DVM_VM_THREADS * 16) + (ib & 3) * 4, 0, 0);
    } else if (op == DVM_OP_STS) {
      push(DVM_LK_W0(DVM_LK_STS, 0, ia, tag), DVM_HDR_WORDS + 2 * nt + ib * DVM_OPD_WORDS, 0, 0);
    } else if (op == DVM_OP_BCS) {
      push(DVM_LK_W0(DVM_LK_BCS, 0, ia, 0), 0, 0, 0);
    } else if (op == DVM_OP_SOP) {
      push(DVM_LK_W0(DVM_LK_SOP, ib, ia, tag), body[pc + 1], len > 2 ? body[pc + 2] : 0, len > 3 ? body[pc + 3] : 0);
    } else if (op >= DVM_OP_CMP && op <= DVM_OP_CMP + DVM_C_NE) {
      // Table 1, Cmp against an fp32 image, a temporary or the accumulator itself (bf16 images, Pow: general interpreter)
      if (ia == DVM_REG_ACC) {
        push(DVM_LK_W0(DVM_LK_CMP, op - DVM_OP_CMP, 3, 0), 0, 0, 0);
      } else {
        const uint32_t oy = opw(ia, ib, &kind);
        if (kind == 0) return 0;
        push(DVM_LK_W0(DVM_LK_CMP, op - DVM_OP_CMP, kind, 0), oy, 0, 0);
      }
    } else if (op == DVM_OP_SEL + 3) {
      push(DVM_LK_W0(DVM_LK_SEL, 3, 0, 0), body[pc + 1], body[pc + 2], 0);
    } else if (op >= DVM_OP_SEL && op < DVM_OP_SEL + 3) {
      int kp = 0, kq = 0;
      const uint32_t op_ = opw(ia, (ib >> 6) & 1, &kp), oq = opw(ib & 0x3f, (ib >> 7) & 1, &kq);
      if (kp == 0 || kq == 0) return 0;
      push(DVM_LK_W0(DVM_LK_SEL, op - DVM_OP_SEL, (uint32_t)kp | ((uint32_t)kq << 2), 0), op_, oq, 0);
    } else if (op == DVM_OP_NOP) {
    } else {
      return 0;  // Pow, IsFinite, Cmp / Select on bf16 images: not the lean interpreter's
    }
    pc += len;
  }
  // ---- fusions over neighbouring records ----
  auto hid = [&](uint32_t i) { return rec[i].w[0] & 0xffu; };
  auto sub = [&](uint32_t i) { return (rec[i].w[0] >> 8) & 0xffu; };
  uint32_t m = 0;
  for (uint32_t i = 0; i < n; ++i) {
    Rec r = rec[i];
    const uint32_t h = r.w[0] & 0xffu;
    if (i + 1 < n) {
      const uint32_t h2 = hid(i + 1), s2 = sub(i + 1);
      // ACC = L[x] ; ACC = ACC op L[y], both bf16 images  ->  LD2 (fp32 pairs stay two records: their raw words fill the registers)
      if (h == DVM_LK_LDA_BF16 && h2 == DVM_LK_BIN_BF16) {
        if ((s2 == DVM_A_ADD || s2 == DVM_A_SUB || s2 == DVM_A_RSUB || s2 == DVM_A_MUL) && !(rec[i + 1].w[0] >> 24)) {
          r.w[0] = DVM_LK_W0(DVM_LK_LD2_BF16, s2, 0, 0);
          r.w[2] = rec[i + 1].w[1];
          ++i;
          // ... followed by a multiplication by an immediate
          if (i + 1 < n && hid(i + 1) == DVM_LK_FMA && sub(i + 1) == 0 && rec[i + 1].w[2] == f2u(neg_zero)) {
            r.w[0] |= 1u << 24;
            r.w[3] = rec[i + 1].w[1];
            ++i;
          }
          rec[m++] = r;
          continue;
        }
      }
      // multiply by an immediate, then add an immediate  ->  one multiply-add
      if (h == DVM_LK_FMA && sub(i) == 0 && r.w[2] == f2u(neg_zero) && h2 == DVM_LK_FMA && s2 == 0 && rec[i + 1].w[1] == f2u(one)) {
        r.w[2] = rec[i + 1].w[2];
        ++i;
        rec[m++] = r;
        continue;
      }
      // ACC = ACC * S[a] ; ACC = ACC * L[y]  ->  BIN with a pre-multiplier
      if (h == DVM_LK_FMA && sub(i) == 1 && r.w[2] == f2u(neg_zero) && (h2 == DVM_LK_BIN_BF16 || h2 == DVM_LK_BIN_F32) &&
          s2 == DVM_A_MUL && !(rec[i + 1].w[0] >> 24)) {
        Rec q = rec[i + 1];
        q.w[0] |= (1u + ((r.w[0] >> 16) & 0xffu)) << 24;
        ++i;
        rec[m++] = q;
        continue;
      }
    }
    rec[m++] = r;
  }
  n = m;
  // the records start at a word index = 0 mod 4 of the parameter block (16-byte aligned in the kernel's parameter space)
  uint32_t rec0 = head;
  while ((at + rec0) % 4 != 0) ++rec0;
  if (rec0 + 4 * (n + 1) > max_words) return 0;
  for (uint32_t i = head; i < rec0; ++i) dst[i] = 0;
  for (uint32_t i = 0; i < n; ++i) memcpy(dst + rec0 + 4 * i, rec[i].w, 16);
  uint32_t* end = dst + rec0 + 4 * n;
  end[0] = DVM_LK_W0(DVM_LK_END, 0, 0, 0); end[1] = end[2] = end[3] = 0;
  ++n;
  // Header words the device never reads carry what the lean interpreter wants ready: the offset of the records
  // (magic word) and the multipliers that divide a row index by the two inner outer-dim sizes.
  auto magic = [](uint32_t d, uint32_t* mult, uint32_t* l) {
    uint32_t lg = 0;
    while (lg < 32 && ((uint64_t)1 << lg) < d) ++lg;
    *l = lg;
    *mult = d ? (uint32_t)((((uint64_t)1 << 32) * (((uint64_t)1 << lg) - d)) / d + 1) : 0;
  };
  dst[DVM_H_MAGIC] = rec0;
  magic(src[DVM_H_OUTER0], &dst[DVM_H_KERNEL_TYPE], &dst[DVM_H_CODE_WORDS]);
  magic(src[DVM_H_OUTER1], &dst[DVM_H_N_TILES], &dst[DVM_H_TOTAL_WORDS]);
  return rec0 + 4 * n;
}

// Results that tiles combine atomically start from the operation's identity.
__global__ void dvm_fill_kernel(uint32_t* p, uint32_t n, uint32_t bits) {
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) p[i] = bits;
}

int prefill_combined(const uint32_t* code, void* const* tensors, cudaStream_t stream) {
  const uint32_t counts = code[DVM_H_COUNTS];
  const uint32_t nt = counts & 0xff, n_opd = (counts >> 16) & 0xff;
  const uint32_t* ot = code + DVM_HDR_WORDS + 2 * nt;
  for (uint32_t o = 0; o < n_opd; ++o) {
    const uint32_t info = ot[o * DVM_OPD_WORDS + DVM_OPD_INFO], comb = (info >> 26) & 3u;
    if (!comb) continue;
    const uint32_t n = ot[o * DVM_OPD_WORDS + DVM_OPD_FILL];
    if (n == 0) continue;
    const uint32_t bits = comb == 1 ? 0u : (comb == 2 ? 0xff800000u : 0x7f800000u);  // 0, -inf, +inf
    const int blocks = (int)((n + 255u) / 256u < 1184u ? (n + 255u) / 256u : 1184u);
    dvm_fill_kernel<<<blocks, 256, 0, stream>>>(static_cast<uint32_t*>(tensors[info & 0xff]), n, bits);
    DVM_CUDA(cudaGetLastError());
    dvm_count_launch();
  }
  return DVM_OK;
}

int prefill_all(int n_programs, const void* const* codes, void* const* const* tensors, cudaStream_t stream) {
  for (int i = 0; i < n_programs; ++i) {
    const uint32_t* c = (const uint32_t*)codes[i];
    if (!((c[DVM_H_GEOM] >> 24) & DVM_F_VIEWS)) continue;
    int st = prefill_combined(c, tensors[i], stream);
    if (st != DVM_OK) return st;
  }
  return DVM_OK;
}

// Starts one interpreter variant on `grid` CTAs.
int launch_variant(const DvmVmVariant* v, const void* params, int grid, size_t smem, cudaStream_t stream) {
  t_last_variant = v;
  DVM_CUDA(v->launch(params, grid, smem, stream));
  dvm_count_launch();
  return DVM_OK;
}

// The variant a launch needs: 24 elements per thread exist as the one-program basic variant only.
const DvmVmVariant* pick_variant(int V, bool large, bool single, int ext, bool levels, int lean, bool heavy) {
  if (levels) single = false;
  return dvm_vm_find_variant(V, large, single, ext, levels, lean, heavy);
}

// What decides between the lean kernel and the general one, read off a placed program (tensor addresses known):
//   wrap  -- a row may fill the tile's whole capacity while its chunks are shifted by a misaligned row start, so
//            that its last columns wrap around into the head slots: only the general kernel does that;
//   heavy -- a tile-class unary function that only the HEAVY variants of the lean kernel carry.
void program_traits(const uint32_t* w, void* const* tensors, bool* wrap, bool* heavy) {
  const uint32_t geom = w[DVM_H_GEOM];
  uint32_t flags = geom >> 24;
  const uint32_t lgG = geom & 0xff, W = (geom >> 8) & 0xff, V = w[DVM_H_LOCAL] >> 24;
  const uint32_t counts = w[DVM_H_COUNTS];
  const uint32_t* ot = w + DVM_HDR_WORDS + 2 * (counts & 0xff);
  if ((flags & DVM_F_ALIGNED) && w[DVM_H_PRIMARY] != 0xffffffffu &&
      (((uintptr_t)tensors[ot[w[DVM_H_PRIMARY] * DVM_OPD_WORDS] & 0xff]) & 15))
    flags &= ~(uint32_t)DVM_F_ALIGNED;  // (what place_program does to the placed copy)
  if (!(flags & DVM_F_ALIGNED) && (uint64_t)w[DVM_H_COL_TILE] + W - 1 > ((uint64_t)V << lgG)) *wrap = true;
  const uint32_t* body = ot + ((counts >> 16) & 0xff) * DVM_OPD_WORDS + ((geom >> 16) & 0xff);
  const uint32_t end = w[DVM_H_CODE_WORDS];
  for (uint32_t pc = w[DVM_H_LOAD_WORDS]; pc < end;) {
    const uint32_t op = DVM_INSN_OP(body[pc]), len = DVM_INSN_LEN(body[pc]);
    if (op >= DVM_OP_UN && op < DVM_OP_UN + DVM_U_NUN) {
      const uint32_t u = op - DVM_OP_UN;
      if (u == DVM_U_SQRT || u == DVM_U_LOG || u == DVM_U_ERF || u == DVM_U_FLOOR || u == DVM_U_ROUND || u == DVM_U_TANH ||
          u == DVM_U_TRUNC_I32 || u == DVM_U_TRUNC_U8) *heavy = true;
    }
    if (op >= DVM_OP_ACT && op < DVM_OP_ACT + DVM_ACT_N) *heavy = true;
    if (op >= DVM_OP_CMP && op <= DVM_OP_SEL + 3) *heavy = true;  // (Cmp / Select: in the HEAVY variants of the lean kernel)
    pc += len ? len : 1;
  }
}

// Phases of a phased program (rows longer than a tile run in phases over their column blocks: DVM_OP_PHASE), 0 for the rest.
uint32_t program_phases(const uint32_t* w) {
  const uint32_t counts = w[DVM_H_COUNTS], geom = w[DVM_H_GEOM];
  const uint32_t* body = w + DVM_HDR_WORDS + 2 * (counts & 0xff) + ((counts >> 16) & 0xff) * DVM_OPD_WORDS + ((geom >> 16) & 0xff);
  return w[DVM_H_LOAD_WORDS] < w[DVM_H_CODE_WORDS] ? DVM_PHASES_OF(body[w[DVM_H_LOAD_WORDS]]) : 0u;
}

// ---- debug mode (environment variable DVM_DEBUG=1) ----
// Before the interpreter starts, one thread on the DEVICE walks the parameter block as it arrived there: the
// directory, every program's header, tables and instructions -- tensor pointers present and aligned to their
// element type, register / operand / tensor-slot indices inside their tables, instruction lengths inside the
// code body.  A failed check sets the status word (the launch is then not made); nothing is dereferenced.
bool debug_mode() {
  static const bool on = getenv("DVM_DEBUG") && atoi(getenv("DVM_DEBUG")) != 0;
  return on;
}
template <int PW>
__global__ void dvm_debug_check_kernel(const __grid_constant__ dvm::VMParams<PW> prm) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  bool ok = prm.n_programs >= 1 && prm.n_words <= (uint32_t)PW;
  const uint32_t n = prm.n_programs;
  for (uint32_t i = 0; ok && i < n; ++i) {
    const uint32_t at = prm.words[i];
    if (at + DVM_HDR_WORDS > prm.n_words) { ok = false; break; }
    const uint32_t* w = prm.words + at;
    const uint32_t counts = w[DVM_H_COUNTS], geom = w[DVM_H_GEOM];
    const uint32_t nt = counts & 0xff, n_opd = (counts >> 16) & 0xff, n_lregs = (geom >> 16) & 0xff;
    const uint32_t body = w[DVM_H_CODE_WORDS], load_words = w[DVM_H_LOAD_WORDS];
    const uint32_t total = DVM_HDR_WORDS + 2 * nt + DVM_OPD_WORDS * n_opd + n_lregs + body;
    if (w[DVM_H_MAGIC] != DVM_MAGIC || w[DVM_H_KERNEL_TYPE] != DVM_KERNEL_VEC || total != w[DVM_H_TOTAL_WORDS] ||
        at + total > prm.n_words || nt > DVM_MAX_TENSORS || n_opd > DVM_MAX_OPERANDS || n_lregs > DVM_MAX_LREGS || load_words > body) {
      ok = false;
      break;
    }
    const uint32_t* ot = w + DVM_HDR_WORDS + 2 * nt;
    const uint32_t* lt = ot + n_opd * DVM_OPD_WORDS;
    const uint32_t* code = lt + n_lregs;
    for (uint32_t o = 0; ok && o < n_opd; ++o) {
      const uint32_t info = ot[o * DVM_OPD_WORDS], slot = info & 0xff, dt = (info >> 8) & 0xff;
      if (slot >= nt || dt > DVM_DT_I32) { ok = false; break; }
      const unsigned long long p = ((unsigned long long)w[DVM_HDR_WORDS + 2 * slot + 1] << 32) | w[DVM_HDR_WORDS + 2 * slot];
      if (p == 0 || (p & ((1ull << DVM_DT_LG_ES(dt)) - 1))) ok = false;
    }
    for (uint32_t k = 0; ok && k < (w[DVM_H_LOCAL] & 0xff); ++k)
      if (k >= n_lregs || (lt[k] >> 24) >= n_opd) ok = false;
    for (uint32_t pc = 0; ok && pc < body;) {
      const uint32_t w0 = code[pc], op = DVM_INSN_OP(w0), len = DVM_INSN_LEN(w0), a = DVM_INSN_A(w0), b = DVM_INSN_B(w0);
      if (len == 0 || pc + len > body || op >= DVM_OP_LAST) { ok = false; break; }
      if (op == DVM_OP_LDG && ((a & 0x7f) >= n_lregs || b >= n_opd)) ok = false;
      if ((op == DVM_OP_STG || op == DVM_OP_LDS || op == DVM_OP_STS) && b >= n_opd) ok = false;
      if ((op == DVM_OP_LDA || op == DVM_OP_STA) && a >= n_lregs) ok = false;
      if (((op >= DVM_OP_BIN && op < DVM_OP_BIN + DVM_A_NBIN) || (op >= DVM_OP_CMP && op < DVM_OP_CMP + DVM_C_NCMP)) &&
          a != DVM_REG_ACC && a >= n_lregs)
        ok = false;
      if (((op >= DVM_OP_LD2 && op < DVM_OP_LD2 + DVM_A_NBIN) || (op >= DVM_OP_SEL && op < DVM_OP_SEL + 3)) &&
          (a >= n_lregs || (b & 0x3f) >= n_lregs))
        ok = false;
      if (((op >= DVM_OP_BINS && op < DVM_OP_BINS + DVM_A_NBIN) || (op >= DVM_OP_RED && op < DVM_OP_RED + DVM_R_NRED) ||
           op == DVM_OP_BCS || op == DVM_OP_LSS || op == DVM_OP_SOP) && a >= DVM_MAX_SREGS)
        ok = false;
      if ((pc < load_words) != (op == DVM_OP_LDG || op == DVM_OP_LDS)) ok = false;
      pc += len;
    }
  }
  if (!ok) atomicMax(prm.status, (unsigned int)dvm::ST_BAD_CODE);
}

// Debug mode, before the interpreter launch: the device-side check of the placed block, then a synchronisation; returns
// the status the device reported (and clears it).
template <int PW>
int debug_check(const dvm::VMParams<PW>& P, cudaStream_t stream) {
  dvm_debug_check_kernel<PW><<<1, 32, 0, stream>>>(P);
  DVM_CUDA(cudaGetLastError());
  dvm_count_launch();
  int status = DVM_OK;
  const int st = dvm_last_device_status((void*)stream, &status);
  return st != DVM_OK ? st : status;
}

static_assert(offsetof(dvm::VMParams<PW_SMALL>, words) % 16 == 0 && offsetof(dvm::VMParams<PW_LARGE>, words) % 16 == 0,
              "linked records are loaded as 16-byte vectors of the parameter space");
thread_local dvm::VMParams<PW_LARGE> t_large;  // 32 KB, reused by every launch of the thread

// Writes the directory and the programs of a launch into the parameter block P.  `linked`: in the linked form
// of the lean interpreter; returns DVM_ERR_UNSUPPORTED when some program cannot be linked or the linked forms
// do not fit (the caller then places the plain forms for the general interpreter).
int place_all(dvm::VMParams<PW_LARGE>& P, int n_programs, const void* const* codes, void* const* const* tensors,
              const int* n_tensors, const int* level, bool linked, uint32_t* words_used) {
  const uint32_t dir = (level ? 3 : 2) * (uint32_t)n_programs + 1;
  uint32_t pos = dir, tb = 0, level_start = 0;
  for (int i = 0; i < n_programs; ++i) {
    const uint32_t* c = (const uint32_t*)codes[i];
    if (pos + c[DVM_H_TOTAL_WORDS] > (uint32_t)PW_LARGE) return linked ? DVM_ERR_UNSUPPORTED : DVM_ERR_TOO_LARGE;
    P.words[i] = pos;
    P.words[n_programs + i] = tb;
    if (level) {
      if (i > 0 && level[i] != level[i - 1]) level_start = tb;  // every tile before this one belongs to a lower level
      P.words[2 * n_programs + 1 + i] = level_start;
    }
    int st = place_program(P.words + pos, c, tensors[i], n_tensors[i]);
    if (st != DVM_OK) return st;
    uint32_t used = c[DVM_H_TOTAL_WORDS];
    if (linked) {
      used = dvm_link_program(P.words + pos, pos, (uint32_t)PW_LARGE - pos, c, tensors[i]);
      if (used == 0) return DVM_ERR_UNSUPPORTED;
    }
    pos += used;
    tb += c[DVM_H_N_TILES];
  }
  P.words[2 * n_programs] = tb;
  *words_used = pos;
  return DVM_OK;
}

// Whether every input of a program is aligned like the tile's chunks: the tensor on a 16-byte boundary, its rows
// (and column blocks; for a row-by-row copied input its outer strides) a whole number of 16-byte units, a chunk of
// it 16 bytes or more.  Then no read of an image needs realigning (the lean interpreter has a build without that code).
bool program_all_aligned(const uint32_t* c, void* const* tensors) {
  const uint32_t geom = c[DVM_H_GEOM];
  if (!((geom >> 24) & DVM_F_ALIGNED)) return false;
  const uint32_t counts = c[DVM_H_COUNTS], nt = counts & 0xff, n_opd = (counts >> 16) & 0xff;
  const uint32_t* ot = c + DVM_HDR_WORDS + 2 * nt;
  const uint32_t* lt = ot + n_opd * DVM_OPD_WORDS;
  const uint32_t n_inr = c[DVM_H_LOCAL] & 0xff, W = (geom >> 8) & 0xff;
  const uint64_t C = c[DVM_H_COLS], ctile = c[DVM_H_COL_TILE], cb = c[DVM_H_COL_BLOCKS];
  for (uint32_t k = 0; k < n_inr; ++k) {
    const uint32_t mode = (lt[k] >> 16) & 0xf, info = ot[(lt[k] >> 24) * DVM_OPD_WORDS];
    const uint32_t dt = (info >> 8) & 0xff;
    const uint64_t es = (uint64_t)1 << DVM_DT_LG_ES(dt);
    if (((uintptr_t)tensors[info & 0xff]) & 15) return false;
    if (W * es < 16) return false;  // (a chunk of 4 bf16 elements is 8 bytes)
    if (cb > 1 && (ctile * es) % 16) return false;
    if (mode == DVM_LM_BLOCK) {
      if ((C * es) % 16) return false;
    } else if (mode == DVM_LM_ROWS) {  // a row copied on its own starts wherever the outer strides put it
      const uint32_t* d = ot + (lt[k] >> 24) * DVM_OPD_WORDS;
      for (int q = 0; q < 3; ++q)
        if (((uint64_t)d[DVM_OPD_STRIDE0 + 2 * q] * es) % 16 || d[DVM_OPD_STRIDE0 + 2 * q + 1]) return false;
    } else if (mode != DVM_LM_BCAST && mode != DVM_LM_BCAST_TILE) {
      return false;
    }
  }
  return true;
}

// `level` (may be NULL): level[i] of program i, non-decreasing; a program reads what programs of lower levels store.
// `tile_begin`, `tile_end` (one-program launches without a queue; 0, 0 = all): the range of tiles to run.
int launch_vec(int n_programs, const void* const* codes, void* const* const* tensors, const int* n_tensors,
               bool use_queue, const int* level, cudaStream_t stream, uint32_t tile_begin = 0, uint32_t tile_end = 0) {
  // A program that asks for a single tile slot (DVM_F_ONE_SLOT), launched on its own: the lean interpreter runs
  // it with one slot; on the general interpreter the variant with level waits does (every tile held back until
  // the CTA's previous tile is done, nothing waited for).
  bool one_slot = n_programs == 1 && !level &&
                  ((((const uint32_t*)codes[0])[DVM_H_GEOM] >> 24) & DVM_F_ONE_SLOT) != 0;
  static const int kOneLevel[1] = {0};
  static const int kNoLevels[DVM_MAX_STACK] = {0};
  // stacked launches with one tile slot per CTA (dvm_set_stacked_one_slot): every program on level 0, every tile's
  // loads held back until the CTA's previous tile is done -- twice the tile size fits two CTAs per SM
  if (g_stacked_one_slot && use_queue && !level && n_programs >= 1) { one_slot = true; level = kNoLevels; }
  const bool queue_asked = use_queue;
  // directory: [program word offsets (n)][tile prefix sums (n+1)][tiles before the program's level (n, with levels)]
  uint32_t dir = (level ? 3 : 2) * (uint32_t)n_programs + 1;
  uint64_t need = dir;
  uint64_t total_tiles = 0;
  uint32_t units = 0;
  uint32_t row_tiles = 0;
  bool phased_basic = false;
  int V = 0;
  int ext = 0;  // the extension level the launch needs: 1 Cmp / Select / Pow / IsFinite, 2 also views
  for (int i = 0; i < n_programs; ++i) {
    const uint32_t* c = (const uint32_t*)codes[i];
    need += c[DVM_H_TOTAL_WORDS];
    total_tiles += c[DVM_H_N_TILES];
    if ((c[DVM_H_LOCAL2] >> 16) > units) units = c[DVM_H_LOCAL2] >> 16;
    const int v = (int)(c[DVM_H_LOCAL] >> 24);
    if (((c[DVM_H_GEOM] >> 24) & DVM_F_EXT_ISA) && ext < 1) ext = 1;
    if ((c[DVM_H_GEOM] >> 24) & DVM_F_VIEWS) ext = 2;
    if (V && v != V) return DVM_ERR_INVALID_ARG;  // one kernel variant per launch: same elements per thread
    V = v;
    const uint32_t phases = program_phases(c);
    if (phases) {
      // a phased program: a CTA walks the tiles of a row in order -- a launch of its own, without a work queue;
      // the views variant of the interpreter carries the phase logic
      if (n_programs != 1 || use_queue || level || tile_end) return DVM_ERR_UNSUPPORTED;
      if (total_tiles > 0x7fffffffull) return DVM_ERR_TOO_LARGE;
      row_tiles = phases * c[DVM_H_COL_BLOCKS];
      phased_basic = ext == 0;  // nothing else asks for the general interpreter: the lean one has a phased variant
      ext = 2;
    }
  }
  if (need > PW_LARGE || total_tiles > 0xffffffffull) return DVM_ERR_TOO_LARGE;
  if (tile_end) {  // a range of the program's tiles
    if (n_programs != 1 || use_queue || level || tile_begin > tile_end || tile_end > total_tiles) return DVM_ERR_INVALID_ARG;
    total_tiles = tile_end;
  } else {
    tile_begin = 0;
  }
  if (total_tiles == tile_begin) return DVM_OK;

  DvmDeviceInfo dev;
  int st = dvm_device_state(&dev);
  if (st != DVM_OK) return st;

  dvm::VMParams<PW_LARGE>& P = t_large;
  bool wrap = false, heavy = false;
  for (int i = 0; i < n_programs; ++i) {
    const uint32_t nt = ((const uint32_t*)codes[i])[DVM_H_COUNTS] & 0xff;
    if ((uint32_t)n_tensors[i] != nt) return DVM_ERR_INVALID_ARG;
    for (uint32_t q = 0; q < nt; ++q) if (!tensors[i][q]) return DVM_ERR_INVALID_ARG;
    program_traits((const uint32_t*)codes[i], tensors[i], &wrap, &heavy);
  }
  // (launches with a work queue run on the general interpreter unless asked otherwise: measured faster there)
  int lean = (ext <= 1 && !level && !wrap && !(one_slot && queue_asked) && (!queue_asked || g_use_lean >= 2)) ? (g_use_lean ? 1 : 0) : 0;
  // a phased program of the basic instruction set: the lean interpreter's phased variant (lean = 2), when the
  // library has one for these elements per thread
  if (phased_basic && !wrap && g_use_lean && dvm_vm_find_variant(V, false, true, 0, false, 2, heavy)) lean = 2;
  if (debug_mode()) lean = 0;  // the bytecode itself travels to the device, where the check kernel reads it
  uint32_t pos = 0;
  st = lean ? place_all(P, n_programs, codes, tensors, n_tensors, level, true, &pos) : DVM_ERR_UNSUPPORTED;
  if (st == DVM_ERR_UNSUPPORTED) {
    lean = 0;
    if (one_slot && !level) { level = kOneLevel; use_queue = true; }
    if (tile_end && use_queue) return DVM_ERR_UNSUPPORTED;  // (tile ranges exist for launches without a work queue)
    st = place_all(P, n_programs, codes, tensors, n_tensors, level, false, &pos);
  }
  if (st != DVM_OK) return st;
  P.n_programs = (uint32_t)n_programs;
  P.total_tiles = (uint32_t)total_tiles;
  P.n_words = pos;
  P.use_queue = use_queue ? 1u : 0u;
  P.levels = one_slot ? 2u : (level ? 1u : 0u);
  P.tile_begin = tile_begin;
  P.row_tiles = row_tiles;
  P.status = dev.scratch;
  P.queue = dev.scratch + 8 + 4 * dev.queue_slot;

  const bool large = pos > PW_SMALL;
  const size_t smem = ((one_slot ? 1 : 2) * (size_t)units + 1) * DVM_LOCAL_UNIT;  // one spare unit, two tile slots (or one)
  P.slot_bytes = one_slot ? 0u : units * DVM_LOCAL_UNIT;
  if (smem > kMaxDynSmem) return DVM_ERR_TOO_LARGE;
  const bool single = n_programs == 1 && !use_queue;
  const DvmVmVariant* variant = pick_variant(V, large, single, lean ? 0 : ext, level != nullptr, lean, heavy);
  if (one_slot && variant && 3 * (smem + 9600) <= 233472) {
    // one tile slot per CTA, and three such CTAs fit an SM: the kernel compiled for three (where the library has it)
    const DvmVmVariant* v3 = dvm_vm_find_variant(V, large, variant->single != 0, variant->ext, variant->levels != 0, variant->lean,
                                                 variant->heavy != 0, 3);
    if (v3) variant = v3;
  }
  if (lean == 1 && single && one_slot && variant && variant->ctas == 3) {
    // one program with one tile slot on the build for three CTAs: its build for aligned programs
    const uint32_t* c0 = (const uint32_t*)codes[0];
    const DvmVmVariant* v9 = program_all_aligned(c0, tensors[0]) ? dvm_vm_find_variant(V, large, true, 0, false, 9, heavy, 3) : nullptr;
    if (v9) variant = v9;
  }
  if (lean == 1 && single && !one_slot && variant) {
    // one program with two tile slots: the build without the one-slot path
    const uint32_t* c0 = (const uint32_t*)codes[0];
    const bool dense = !((c0[DVM_H_GEOM] >> 24) & (DVM_F_LOADS_BY_ROW | DVM_F_OUTER_DIMS)) && ((c0[DVM_H_LOCAL] >> 16) & 0xff) == 0;
    const bool aligned = program_all_aligned(c0, tensors[0]);
    // every row fills the slots of the threads that hold it: columns = threads per row x elements per thread
    const bool full = c0[DVM_H_COL_BLOCKS] == 1 && c0[DVM_H_LAST_ROW_COLS] == c0[DVM_H_COLS] &&
                      c0[DVM_H_COLS] == ((uint32_t)V << (c0[DVM_H_GEOM] & 0xff));
    const DvmVmVariant* v2 = (aligned && full) ? dvm_vm_find_variant(V, large, true, 0, false, dense ? 7 : 8, heavy) : nullptr;
    if (!v2 && aligned) v2 = dvm_vm_find_variant(V, large, true, 0, false, dense ? 5 : 6, heavy);
    if (!v2 && dense) v2 = dvm_vm_find_variant(V, large, true, 0, false, 4, heavy);
    if (!v2) v2 = dvm_vm_find_variant(V, large, true, 0, false, 3, heavy);
    if (v2) variant = v2;
  }
  if (!variant) return DVM_ERR_UNSUPPORTED;  // (24 elements per thread: encoded for a launch of its own on the basic variant)
  int occ = 0;
  st = dvm_occupancy(variant, smem, &occ);
  if (st != DVM_OK) return st;
  uint64_t slots = (uint64_t)dev.sm_count * occ;
  const uint64_t run_tiles = row_tiles ? total_tiles / row_tiles : total_tiles - tile_begin;  // (phased: whole rows per CTA)
  int grid = (int)(run_tiles < slots ? run_tiles : slots);
  // Everything is placed and checked: only now touch the caller's memory.  Results that tiles combine
  // atomically are filled with their identity (one small kernel per such output), then the interpreter starts.
  st = prefill_all(n_programs, codes, tensors, stream);
  if (st != DVM_OK) return st;
  if (!large) {
    dvm::VMParams<PW_SMALL> S;
    memcpy(&S, &P, offsetof(dvm::VMParams<PW_SMALL>, words) + (size_t)pos * 4);
    if (debug_mode()) {
      st = debug_check(S, stream);
      if (st != DVM_OK) return st;
      st = launch_variant(variant, &S, grid, smem, stream);
      if (st != DVM_OK) return st;
      int status = DVM_OK;
      st = dvm_last_device_status((void*)stream, &status);
      return st != DVM_OK ? st : status;
    }
    return launch_variant(variant, &S, grid, smem, stream);
  }
  if (debug_mode()) {
    st = debug_check(P, stream);
    if (st != DVM_OK) return st;
    st = launch_variant(variant, &P, grid, smem, stream);
    if (st != DVM_OK) return st;
    int status = DVM_OK;
    st = dvm_last_device_status((void*)stream, &status);
    return st != DVM_OK ? st : status;
  }
  return launch_variant(variant, &P, grid, smem, stream);
}

}  // namespace

extern "C" int dvm_launch_checked(const void* code, size_t code_size, void* const* tensors, const size_t* tensor_bytes,
                                  int n_tensors, void* cuda_stream) {
  if (!code || !tensors || !tensor_bytes || n_tensors < 0 || n_tensors > DVM_MAX_TENSORS) return DVM_ERR_INVALID_ARG;
  int64_t need[DVM_MAX_TENSORS];
  int st = dvm_tensor_extents(code, code_size, need, n_tensors);
  if (st != DVM_OK) return st;
  for (int i = 0; i < n_tensors; ++i)
    if ((int64_t)tensor_bytes[i] < need[i]) return DVM_ERR_BUFFER_TOO_SMALL;
  return dvm_launch(code, code_size, tensors, n_tensors, cuda_stream);
}

extern "C" int dvm_launch(const void* code, size_t code_size, void* const* tensors, int n_tensors,
                          void* cuda_stream) {
  if (!code || !tensors) return DVM_ERR_INVALID_ARG;
  int st = dvm_verify(code, code_size);
  if (st != DVM_OK) return st;
  const uint32_t* w = (const uint32_t*)code;
  if (w[DVM_H_KERNEL_TYPE] == DVM_KERNEL_MATMUL)
    return dvm_launch_matmul(w, code_size / 4, tensors, n_tensors, (cudaStream_t)cuda_stream);
  const void* codes[1] = {code};
  void* const* tl[1] = {tensors};
  return launch_vec(1, codes, tl, &n_tensors, false, nullptr, (cudaStream_t)cuda_stream);
}

extern "C" int dvm_launch_stacked(int n_programs, const void* const* codes, const size_t* code_sizes,
                                  void* const* const* tensors, const int* n_tensors, void* cuda_stream) {
  if (n_programs < 0 || (n_programs > 0 && (!codes || !code_sizes || !tensors || !n_tensors)))
    return DVM_ERR_INVALID_ARG;
  if (n_programs == 0) return DVM_OK;
  if (n_programs > DVM_MAX_STACK) return DVM_ERR_TOO_LARGE;
  for (int i = 0; i < n_programs; ++i) {
    if (!codes[i] || !tensors[i]) return DVM_ERR_INVALID_ARG;
    int st = dvm_verify(codes[i], code_sizes[i]);
    if (st != DVM_OK) return st;
    // only vector meta-kernels stack (Sec. 5.1: stacking of meta-kernels on the Vector units)
    if (((const uint32_t*)codes[i])[DVM_H_KERNEL_TYPE] != DVM_KERNEL_VEC) return DVM_ERR_UNSUPPORTED;
  }
  return launch_vec(n_programs, codes, tensors, n_tensors, true, nullptr, (cudaStream_t)cuda_stream);
}

extern "C" int dvm_launch_stacked_levels(int n_programs, const void* const* codes, const size_t* code_sizes,
                                         void* const* const* tensors, const int* n_tensors, const int* level,
                                         void* cuda_stream) {
  if (n_programs < 0 || (n_programs > 0 && (!codes || !code_sizes || !tensors || !n_tensors || !level)))
    return DVM_ERR_INVALID_ARG;
  if (n_programs == 0) return DVM_OK;
  if (n_programs > DVM_MAX_STACK) return DVM_ERR_TOO_LARGE;
  for (int i = 0; i < n_programs; ++i) {
    if (!codes[i] || !tensors[i]) return DVM_ERR_INVALID_ARG;
    if (i > 0 && level[i] < level[i - 1]) return DVM_ERR_INVALID_ARG;  // the work queue hands tiles out in level order
    int st = dvm_verify(codes[i], code_sizes[i]);
    if (st != DVM_OK) return st;
    if (((const uint32_t*)codes[i])[DVM_H_KERNEL_TYPE] != DVM_KERNEL_VEC) return DVM_ERR_UNSUPPORTED;
  }
  return launch_vec(n_programs, codes, tensors, n_tensors, true, level, (cudaStream_t)cuda_stream);
}

// dvm_run_host pipelines when the program allows it: every tensor either follows the tiles row block by row block
// (a dense operand: the rows of tile t are one byte range) or is a row vector shared by all rows.  The tiles are then
// cut into chunks; chunk k copies its input rows to the device, runs its tiles and copies its output rows back on
// stream k mod 3 of three library-owned streams, so that the copies of one chunk (PCIe in both directions) overlap
// the execution of another.
namespace {
constexpr int kPipeStreams = 3;
struct PipeStreams { bool ready = false; cudaStream_t s[kPipeStreams]; cudaEvent_t done[kPipeStreams]; cudaEvent_t start; };
PipeStreams g_pipe[MAX_DEVICES];

int pipe_streams(PipeStreams** out) {
  int dev = 0;
  DVM_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEVICES) return DVM_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(g_mu);
  PipeStreams& p = g_pipe[dev];
  if (!p.ready) {
    for (int i = 0; i < kPipeStreams; ++i) {
      DVM_CUDA(cudaStreamCreateWithFlags(&p.s[i], cudaStreamNonBlocking));
      DVM_CUDA(cudaEventCreateWithFlags(&p.done[i], cudaEventDisableTiming));
    }
    DVM_CUDA(cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming));
    p.ready = true;
  }
  *out = &p;
  return DVM_OK;
}

// 0: the tensor follows the tiles (rows of `row_bytes` bytes), 1: a row vector copied whole, -1: neither
int pipe_class(const uint32_t* w, const uint32_t* od, bool is_input, uint64_t* row_bytes) {
  const uint32_t info = od[DVM_OPD_INFO];
  const uint32_t es = 1u << DVM_DT_LG_ES((info >> 8) & 0xff);
  if (((info >> 16) & 0xff) != 1 || od[DVM_OPD_COLSTRIDE] != 1 || ((info >> 26) & 3u)) return -1;
  if ((info >> 25) & 1u) {  // dense: row r starts at element r * C
    *row_bytes = (uint64_t)w[DVM_H_COLS] * es;
    return 0;
  }
  if (is_input && od[DVM_OPD_STRIDE0] == 0 && od[DVM_OPD_STRIDE1] == 0 && od[DVM_OPD_STRIDE2] == 0) return 1;
  return -1;
}
}  // namespace

extern "C" int dvm_run_host(const void* code, size_t code_size, void* const* host_tensors,
                            const size_t* tensor_bytes, int n_tensors, void* staging, size_t staging_bytes,
                            void* cuda_stream) {
  if (!code || !host_tensors || !tensor_bytes || !staging) return DVM_ERR_INVALID_ARG;
  int st = dvm_verify(code, code_size);
  if (st != DVM_OK) return st;
  const uint32_t* w = (const uint32_t*)code;
  const uint32_t counts = w[DVM_H_COUNTS];
  const int nt = counts & 0xff, n_in = (counts >> 8) & 0xff;
  if (n_tensors != nt || nt > DVM_MAX_TENSORS) return DVM_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  void* dev[DVM_MAX_TENSORS];
  size_t off = 0;
  for (int i = 0; i < nt; ++i) {
    dev[i] = (char*)staging + off;
    off += (tensor_bytes[i] + 255) & ~(size_t)255;
  }
  if (off > staging_bytes) return DVM_ERR_BUFFER_TOO_SMALL;

  // ---- can the program be pipelined? ----
  bool pipe = w[DVM_H_KERNEL_TYPE] == DVM_KERNEL_VEC && w[DVM_H_COL_BLOCKS] == 1 && w[DVM_H_N_TILES] >= 8;
  int cls[DVM_MAX_TENSORS];
  uint64_t row_bytes[DVM_MAX_TENSORS];
  if (pipe) {
    const uint32_t n_opd = (counts >> 16) & 0xff;
    const uint32_t* ot = w + DVM_HDR_WORDS + 2 * nt;
    for (int i = 0; i < nt; ++i) cls[i] = -2;  // (a tensor no operand names is not touched)
    for (uint32_t o = 0; o < n_opd && pipe; ++o) {
      const uint32_t* od = ot + o * DVM_OPD_WORDS;
      const int slot = od[DVM_OPD_INFO] & 0xff;
      uint64_t rb = 0;
      const int c = pipe_class(w, od, slot < n_in, &rb);
      if (c < 0 || (cls[slot] != -2 && cls[slot] != c)) pipe = false;
      cls[slot] = c;
      row_bytes[slot] = rb;
    }
    for (int i = 0; i < nt && pipe; ++i) if (cls[i] == -2) pipe = false;
  }
  const uint64_t total_bytes = off;
  if (pipe && total_bytes >= (64u << 20)) {
    PipeStreams* ps = nullptr;
    st = pipe_streams(&ps);
    if (st != DVM_OK) return st;
    const uint32_t n_tiles = w[DVM_H_N_TILES];
    const uint32_t R = (uint32_t)DVM_VM_THREADS >> (w[DVM_H_GEOM] & 0xff);   // rows per tile
    // chunks of about 96 MB over all tensors (measured on the C2 sweep: 12 MB 75 GB/s, 24 MB 83, 48 MB 88, 96 - 128 MB 91,
    // 256 MB 90, 384 MB 87), at least one tile, at most 256 chunks
    uint64_t per_tile = 0;
    for (int i = 0; i < nt; ++i) if (cls[i] == 0) per_tile += row_bytes[i] * R;
    uint32_t chunk_tiles = per_tile ? (uint32_t)((96ull << 20) / per_tile) : n_tiles;
    if (chunk_tiles < 1) chunk_tiles = 1;
    if ((n_tiles + chunk_tiles - 1) / chunk_tiles > 256) chunk_tiles = (n_tiles + 255) / 256;
    // row vectors first, on the caller's stream; the chunk streams start behind them
    for (int i = 0; i < n_in; ++i)
      if (cls[i] == 1 && tensor_bytes[i]) DVM_CUDA(cudaMemcpyAsync(dev[i], host_tensors[i], tensor_bytes[i], cudaMemcpyHostToDevice, stream));
    DVM_CUDA(cudaEventRecord(ps->start, stream));
    for (int k = 0; k < kPipeStreams; ++k) DVM_CUDA(cudaStreamWaitEvent(ps->s[k], ps->start, 0));
    const void* codes[1] = {code};
    void* const* tl[1] = {dev};
    int launched = DVM_OK;
    uint32_t k = 0;
    for (uint32_t t0 = 0; t0 < n_tiles; t0 += chunk_tiles, ++k) {
      const uint32_t t1 = t0 + chunk_tiles < n_tiles ? t0 + chunk_tiles : n_tiles;
      cudaStream_t cs = ps->s[k % kPipeStreams];
      for (int i = 0; i < nt; ++i) {
        if (cls[i] != 0 || i >= n_in) continue;
        const uint64_t b0 = (uint64_t)t0 * R * row_bytes[i];
        uint64_t b1 = (uint64_t)t1 * R * row_bytes[i];
        if (b1 > tensor_bytes[i]) b1 = tensor_bytes[i];
        if (b1 > b0) DVM_CUDA(cudaMemcpyAsync((char*)dev[i] + b0, (const char*)host_tensors[i] + b0, b1 - b0, cudaMemcpyHostToDevice, cs));
      }
      launched = launch_vec(1, codes, tl, &n_tensors, false, nullptr, cs, t0, t1);
      if (launched != DVM_OK) break;
      for (int i = n_in; i < nt; ++i) {
        if (cls[i] != 0) continue;
        const uint64_t b0 = (uint64_t)t0 * R * row_bytes[i];
        uint64_t b1 = (uint64_t)t1 * R * row_bytes[i];
        if (b1 > tensor_bytes[i]) b1 = tensor_bytes[i];
        if (b1 > b0) DVM_CUDA(cudaMemcpyAsync((char*)host_tensors[i] + b0, (const char*)dev[i] + b0, b1 - b0, cudaMemcpyDeviceToHost, cs));
      }
    }
    for (int q = 0; q < kPipeStreams; ++q) {
      DVM_CUDA(cudaEventRecord(ps->done[q], ps->s[q]));
      DVM_CUDA(cudaStreamWaitEvent(stream, ps->done[q], 0));
    }
    DVM_CUDA(cudaStreamSynchronize(stream));
    if (launched == DVM_OK) return DVM_OK;
    if (launched != DVM_ERR_UNSUPPORTED || k != 0) return launched;
    // (the first chunk could not be launched as a range of tiles: nothing ran yet, take the plain way)
  }

  for (int i = 0; i < n_in; ++i)
    if (tensor_bytes[i]) DVM_CUDA(cudaMemcpyAsync(dev[i], host_tensors[i], tensor_bytes[i], cudaMemcpyHostToDevice, stream));
  st = dvm_launch(code, code_size, dev, nt, cuda_stream);
  if (st != DVM_OK) return st;
  for (int i = n_in; i < nt; ++i)
    if (tensor_bytes[i]) DVM_CUDA(cudaMemcpyAsync(host_tensors[i], dev[i], tensor_bytes[i], cudaMemcpyDeviceToHost, stream));
  DVM_CUDA(cudaStreamSynchronize(stream));
  return DVM_OK;
}

// ---- self-test of the bounded waits ----
namespace {
__global__ void dvm_selftest_vm_wait_kernel(unsigned int* status) {
  __shared__ __align__(8) unsigned long long bar;
  const uint32_t b = static_cast<uint32_t>(__cvta_generic_to_shared(&bar));
  if (threadIdx.x == 0) {
    dvm::vm_mbar_init(b, 2);  // two arrivals expected, one ever made: the phase never completes
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    dvm::vm_mbar_arrive(b);
  }
  __syncthreads();
  if (!dvm::vm_mbar_wait(b, 0) && threadIdx.x == 0) atomicMax(status, (unsigned int)dvm::ST_TIMEOUT);
}
// The level wait of dvm_launch_stacked_levels on a counter nobody advances (the status word's neighbour,
// which stays zero): it gives up after its limit.
__global__ void dvm_selftest_level_wait_kernel(unsigned int* status) {
  if (threadIdx.x == 0 && !dvm::vm_wait_tiles_done(status + 1, 1u)) atomicMax(status, (unsigned int)dvm::ST_TIMEOUT);
}
}  // namespace

int dvm_selftest_mm_wait(unsigned int* status, cudaStream_t stream);

extern "C" int dvm_selftest_bounded_wait(int which, void* cuda_stream) {
  DvmDeviceInfo dev;
  int st = dvm_device_state(&dev);
  if (st != DVM_OK) return st;
  if (which == 0) {
    dvm_selftest_vm_wait_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(dev.scratch);
    DVM_CUDA(cudaGetLastError());
    dvm_count_launch();
    return DVM_OK;
  }
  if (which == 1) return dvm_selftest_mm_wait(dev.scratch, (cudaStream_t)cuda_stream);
  if (which == 2) {
    dvm_selftest_level_wait_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(dev.scratch);
    DVM_CUDA(cudaGetLastError());
    dvm_count_launch();
    return DVM_OK;
  }
  return DVM_ERR_INVALID_ARG;
}

extern "C" int dvm_last_device_status(void* cuda_stream, int* status) {
  if (!status) return DVM_ERR_INVALID_ARG;
  DVM_CUDA(cudaStreamSynchronize((cudaStream_t)cuda_stream));
  DvmDeviceInfo dev;
  int st = dvm_device_state(&dev);
  if (st != DVM_OK) return st;
  unsigned int v = 0;
  DVM_CUDA(cudaMemcpy(&v, dev.scratch, 4, cudaMemcpyDeviceToHost));
  if (v) DVM_CUDA(cudaMemset(dev.scratch, 0, 4));
  *status = v == dvm::ST_OK ? DVM_OK : (v == dvm::ST_TIMEOUT ? DVM_ERR_DEVICE_TIMEOUT : DVM_ERR_DEVICE_BAD_CODE);
  return DVM_OK;
}

// ---------------------------------------------------------------------------------------------
// dvm_launch_stacked_noalloc: the stacked launch for callers that must not allocate device memory.
//
// dvm_launch_stacked keeps its work-queue counters in a small buffer that the library obtains with
// cudaMalloc the first time a device is used.  Some callers cannot tolerate that: code running inside a
// memory pool or arena that owns every byte of the device, latency-critical serving loops where a first-use
// cudaMalloc (an implicit device synchronisation) is unacceptable, and sandboxes that forbid the allocator
// outright.  For them the same kernel runs with its queue in the fixed array below, which is part of the
// library image: every GPU that loads the library holds these 256 bytes until the process exits.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int NOALLOC_WORDS = 64;                 // 256 bytes: [0] status word, [2..4] work-queue counters
static __device__ __align__(256) unsigned int dvm_noalloc_scratch[NOALLOC_WORDS];

struct NoAllocDevice {
  unsigned int* scratch = nullptr;  // device address of dvm_noalloc_scratch on this device
  int sm_count = 0;
};
NoAllocDevice g_noalloc[MAX_DEVICES];
std::mutex g_noalloc_mu;

// Once per device, with that device current: resolve the array's device address.  In host code the array's
// name is only a stand-in for the symbol; the address a kernel may use comes from cudaGetSymbolAddress.
int noalloc_device(NoAllocDevice* out) {
  int dev = 0;
  DVM_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEVICES) return DVM_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(g_noalloc_mu);
  NoAllocDevice& d = g_noalloc[dev];
  if (!d.scratch) {
    void* p = nullptr;
    DVM_CUDA(cudaGetSymbolAddress(&p, dvm_noalloc_scratch));
    DVM_CUDA(cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev));
    d.scratch = static_cast<unsigned int*>(p);
  }
  *out = d;
  return DVM_OK;
}

}  // namespace

extern "C" int dvm_launch_stacked_noalloc(int n_programs, const void* const* codes, const size_t* code_sizes,
                                          void* const* const* tensors, const int* n_tensors, void* cuda_stream) {
  if (n_programs < 0 || (n_programs > 0 && (!codes || !code_sizes || !tensors || !n_tensors)))
    return DVM_ERR_INVALID_ARG;
  if (n_programs == 0) return DVM_OK;
  if (n_programs > DVM_NOALLOC_MAX_PROGRAMS) return DVM_ERR_TOO_LARGE;  // beyond the stated maximum
  uint32_t dir = 2 * (uint32_t)n_programs + 1;
  uint64_t need = dir, total_tiles = 0;
  uint32_t units = 0;
  int V = 0;
  int ext = 0;  // the extension level the launch needs: 1 Cmp / Select / Pow / IsFinite, 2 also views
  for (int i = 0; i < n_programs; ++i) {
    if (!codes[i] || !tensors[i]) return DVM_ERR_INVALID_ARG;
    int st = dvm_verify(codes[i], code_sizes[i]);
    if (st != DVM_OK) return st;
    const uint32_t* c = (const uint32_t*)codes[i];
    if (c[DVM_H_KERNEL_TYPE] != DVM_KERNEL_VEC) return DVM_ERR_UNSUPPORTED;
    need += c[DVM_H_TOTAL_WORDS];
    total_tiles += c[DVM_H_N_TILES];
    if ((c[DVM_H_LOCAL2] >> 16) > units) units = c[DVM_H_LOCAL2] >> 16;
    const int v = (int)(c[DVM_H_LOCAL] >> 24);
    if (((c[DVM_H_GEOM] >> 24) & DVM_F_EXT_ISA) && ext < 1) ext = 1;
    if ((c[DVM_H_GEOM] >> 24) & DVM_F_VIEWS) ext = 2;
    if (V && v != V) return DVM_ERR_INVALID_ARG;
    V = v;
    if (program_phases(c)) return DVM_ERR_UNSUPPORTED;  // a phased program is launched on its own (dvm_launch)
  }
  if (need > PW_LARGE || total_tiles > DVM_NOALLOC_MAX_TILES) return DVM_ERR_TOO_LARGE;
  if (total_tiles == 0) return DVM_OK;

  NoAllocDevice dev;
  int st = noalloc_device(&dev);
  if (st != DVM_OK) return st;
  cudaStream_t stream = (cudaStream_t)cuda_stream;

  dvm::VMParams<PW_LARGE>& P = t_large;
  bool wrap = false, heavy = false;
  for (int i = 0; i < n_programs; ++i) {
    const uint32_t nt = ((const uint32_t*)codes[i])[DVM_H_COUNTS] & 0xff;
    if ((uint32_t)n_tensors[i] != nt) return DVM_ERR_INVALID_ARG;
    for (uint32_t q = 0; q < nt; ++q) if (!tensors[i][q]) return DVM_ERR_INVALID_ARG;
    program_traits((const uint32_t*)codes[i], tensors[i], &wrap, &heavy);
  }
  int lean = (ext == 0 && !wrap && g_use_lean >= 2) ? 1 : 0;
  uint32_t pos = 0;
  st = lean ? place_all(P, n_programs, codes, tensors, n_tensors, nullptr, true, &pos) : DVM_ERR_UNSUPPORTED;
  if (st == DVM_ERR_UNSUPPORTED) {
    lean = 0;
    st = place_all(P, n_programs, codes, tensors, n_tensors, nullptr, false, &pos);
  }
  if (st != DVM_OK) return st;
  P.n_programs = (uint32_t)n_programs;
  P.total_tiles = (uint32_t)total_tiles;
  P.n_words = pos;
  P.use_queue = 1u;
  P.levels = 0u;
  P.tile_begin = 0u;
  P.row_tiles = 0u;
  P.status = dev.scratch;
  P.queue = dev.scratch + 2;
  const size_t smem = (2 * (size_t)units + 1) * DVM_LOCAL_UNIT;
  P.slot_bytes = units * DVM_LOCAL_UNIT;
  if (smem > kMaxDynSmem) return DVM_ERR_TOO_LARGE;
  const bool large = pos > PW_SMALL;
  const DvmVmVariant* variant = pick_variant(V, large, false, ext, false, lean, heavy);
  if (!variant) return DVM_ERR_UNSUPPORTED;
  int occ = 0;
  st = dvm_occupancy(variant, smem, &occ);
  if (st != DVM_OK) return st;
  uint64_t slots = (uint64_t)dev.sm_count * occ;
  int grid = (int)(total_tiles < slots ? total_tiles : slots);
  // every call shares the array and it keeps the last call's contents: the queue counters must start at zero
  DVM_CUDA(cudaMemsetAsync(dev.scratch, 0, NOALLOC_WORDS * sizeof(unsigned int), stream));
  st = prefill_all(n_programs, codes, tensors, stream);
  if (st != DVM_OK) return st;
  if (!large) {
    dvm::VMParams<PW_SMALL> S;
    memcpy(&S, &P, offsetof(dvm::VMParams<PW_SMALL>, words) + (size_t)pos * 4);
    return launch_variant(variant, &S, grid, smem, stream);
  }
  return launch_variant(variant, &P, grid, smem, stream);
}
