// The lean variant of the virtual machine (Sec. 4.3, Algorithm 2): it runs every program of the basic
// instruction set (no Cmp / Select / Pow, no views, no level waits, no wrap-around of a row's last columns;
// those run on dvm_vm_kernel) from LINKED code: dvm_launch has turned every bytecode of the compute section
// into a record of four ready-to-use words (dvm_link.h), so the device decodes nothing per tile -- a record is
// one 16-byte load, its handler one branch tree away.
//
// Tile geometry, the two tile slots filled by TMA bulk copies and the load section are those of dvm_vm_kernel
// (see dvm_vm.cuh).  What a tile costs beyond the program's own arithmetic is kept small:
//   * per tile, a thread works out once where its chunks lie (row, shift, the element offset of its first chunk
//     in a dense operand); an operand's address is then the record's offset plus that;
//   * an operand whose rows are aligned differently from the tile's chunks is read as the covering 16-byte
//     vectors and picked apart by a switch on its byte offset -- straight-line code per offset;
//   * slots outside the row are made harmless before a reduction only in the (at most two) 8-slot groups of a
//     thread that the row's head or tail cuts; whole groups outside the row are skipped by predicate;
//   * stores are predicated 16-byte stores per chunk; only cut chunks fall back to element stores;
//   * a reduction carries the scalar multiply-add(-unary) that follows it, exp carries the subtraction of the
//     row maximum before it (fused by the linker);
//   * the heavy unary functions (log, erf, tanh, sqrt, floor, round) exist only in the HEAVY variant, so the
//     hot loop of the programs that do not use them stays small.
#pragma once
#include <type_traits>

#include "dvm_link.h"
#include "dvm_vm.cuh"

#ifndef DVM_LEAN_MIN_CTAS
#define DVM_LEAN_MIN_CTAS 2
#endif

namespace dvm {

__device__ __forceinline__ uint4 lean_lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// A value the compiler must take as it is at this point of this handler.  Several handlers start with the same
// computation on a record's fields (the address of the operand a word names, the load of a per-row scalar); left
// alone, the compiler hoists such common code in front of the dispatch, where EVERY record pays for it (measured:
// a fifth more instructions per tile).  ID makes each use distinct, so nothing can be merged across handlers.
template <int ID>
__device__ __forceinline__ uint32_t lean_opaque(uint32_t v) {
  asm volatile("// handler %1" : "+r"(v) : "n"(ID));
  return v;
}

// bf16 pair in a word -> two floats
__device__ __forceinline__ float2 lean_widen(uint32_t w) {
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

// Raw words of V bf16 elements: V / 8 chunks of 8, chunk j at byte address a + j * vstr.  The chunks of an
// operand aligned like the tile's are 16-byte vectors; otherwise they start E = (a & 15) / 2 elements behind an
// aligned address and are cut out of the two covering vectors (an odd E by byte permutes).
template <int V, int E>
__device__ __forceinline__ void lean_raw_bf16_shift(uint32_t* R, uint32_t b, uint32_t vstr) {
#pragma unroll
  for (int j = 0; j < V / 8; ++j) {
    const uint4 x = lean_lds128(b + j * vstr), y = lean_lds128(b + j * vstr + 16);
    const uint32_t w[8] = {x.x, x.y, x.z, x.w, y.x, y.y, y.z, y.w};
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const int e0 = E + 2 * p;  // first element of the pair, counted in bf16 from b
      R[4 * j + p] = (E % 2 == 0) ? w[e0 / 2] : __byte_perm(w[e0 / 2], w[e0 / 2 + 1], 0x5432);
    }
  }
}
// (AL: the caller knows every operand is aligned like the tile's chunks -- no realignment code at all)
template <int V, bool AL = false>
__device__ __forceinline__ void lean_raw_bf16(uint32_t* R, uint32_t a, uint32_t vstr) {
  const uint32_t mis = AL ? 0u : (a & 15u);
  if (AL || mis == 0) {
#pragma unroll
    for (int j = 0; j < V / 8; ++j) {
      const uint4 v = lean_lds128(a + j * vstr);
      R[4 * j] = v.x; R[4 * j + 1] = v.y; R[4 * j + 2] = v.z; R[4 * j + 3] = v.w;
    }
    return;
  }
  const uint32_t b = a - mis;
  switch (mis >> 1) {
    case 1: lean_raw_bf16_shift<V, 1>(R, b, vstr); break;
    case 2: lean_raw_bf16_shift<V, 2>(R, b, vstr); break;
    case 3: lean_raw_bf16_shift<V, 3>(R, b, vstr); break;
    case 4: lean_raw_bf16_shift<V, 4>(R, b, vstr); break;
    case 5: lean_raw_bf16_shift<V, 5>(R, b, vstr); break;
    case 6: lean_raw_bf16_shift<V, 6>(R, b, vstr); break;
    default: lean_raw_bf16_shift<V, 7>(R, b, vstr); break;
  }
}

// fp32: NV 16-byte vectors per chunk (2 when a chunk has 8 elements, 1 when it has 4); the chunks [J0, J1) of the
// V / (4 NV) chunks of a thread, chunk j at a + j * vstr, starting E words (0..3) behind the aligned address.
// R receives 4 NV words per chunk, from index 0.
template <int NV, int E, int J0, int J1>
__device__ __forceinline__ void lean_raw_f32_shift(uint32_t* R, uint32_t b, uint32_t vstr) {
#pragma unroll
  for (int j = J0; j < J1; ++j) {
    uint32_t w[4 * NV + 4];
#pragma unroll
    for (int q = 0; q < NV + (E ? 1 : 0); ++q) {
      const uint4 x = lean_lds128(b + j * vstr + 16 * q);
      w[4 * q] = x.x; w[4 * q + 1] = x.y; w[4 * q + 2] = x.z; w[4 * q + 3] = x.w;
    }
#pragma unroll
    for (int p = 0; p < 4 * NV; ++p) R[4 * NV * (j - J0) + p] = w[E + p];
  }
}
template <int NV, int J0, int J1, bool AL = false>
__device__ __forceinline__ void lean_raw_f32(uint32_t* R, uint32_t a, uint32_t vstr) {
  if constexpr (AL) {
    lean_raw_f32_shift<NV, 0, J0, J1>(R, a, vstr);
    return;
  }
  const uint32_t mis = a & 15u;
  const uint32_t b = a - mis;
  switch (mis >> 2) {
    case 0: lean_raw_f32_shift<NV, 0, J0, J1>(R, b, vstr); break;
    case 1: lean_raw_f32_shift<NV, 1, J0, J1>(R, b, vstr); break;
    case 2: lean_raw_f32_shift<NV, 2, J0, J1>(R, b, vstr); break;
    default: lean_raw_f32_shift<NV, 3, J0, J1>(R, b, vstr); break;
  }
}

// exp(x) to about 3e-7 relative error (see fast_exp): the product x * log2(e) in two fp32 pieces, the power of
// two from the SFU, a first-order correction -- on pairs, with packed arithmetic.  The residual of an infinite
// argument is NaN; min(r, 1) turns it into 1 (min returns the operand that is a number), so that
// exp(-inf) = 0 + 0 * ln 2 and exp(+inf) = inf + inf * ln 2 come out right.
__device__ __forceinline__ float2 lean_exp2(float2 x) {
  const float2 L2E_HI = make_float2(1.44269502162933349609375f, 1.44269502162933349609375f);
  const float2 L2E_LO = make_float2(1.925963033500011e-8f, 1.925963033500011e-8f);
  const float2 LN2 = make_float2(0.693147182464599609375f, 0.693147182464599609375f);
  const float2 t = __fmul2_rn(x, L2E_HI);
  float2 r = __ffma2_rn(x, L2E_HI, make_float2(-t.x, -t.y));
  r = __ffma2_rn(x, L2E_LO, r);
  r.x = fminf(r.x, 1.0f);
  r.y = fminf(r.y, 1.0f);
  float2 p;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p.x) : "f"(t.x));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p.y) : "f"(t.y));
  return __ffma2_rn(__fmul2_rn(p, r), LN2, p);
}

// x / d for any 32-bit x, from the multiplier m = floor(2^32 (2^l - d) / d) + 1 and l = ceil(log2 d) (sh = l):
// t = mulhi(m, x); q = (t + ((x - t) >> min(l, 1))) >> max(l - 1, 0)
__device__ __forceinline__ uint32_t vm_magic_div(uint32_t x, uint32_t m, uint32_t l) {
  const uint32_t t = __umulhi(m, x);
  return (t + ((x - t) >> (l ? 1u : 0u))) >> (l ? l - 1u : 0u);
}

// exp(x + c) with the product x * log2(e) in one fp32 piece: relative error up to |x + c| * 9e-8 + 2.4e-7 -- what a
// program whose outputs are all bf16 (3.9e-3 per rounding) cannot tell from the longer form.  nc = c * log2(e).
__device__ __forceinline__ float2 lean_exp2_fast(float2 x, float nc) {
  const float2 L2E = make_float2(1.44269502162933349609375f, 1.44269502162933349609375f);
  const float2 t = __ffma2_rn(x, L2E, make_float2(nc, nc));
  float2 p;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p.x) : "f"(t.x));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p.y) : "f"(t.y));
  return p;
}

// PHASED: the variant for phased programs (rows longer than a tile, DVM_OP_PHASE; one program per launch): a CTA takes
// a row through its phases x column blocks in order; everything it adds is behind `if constexpr (PHASED)`.
// CTAS: resident CTAs per SM the kernel is compiled for (2; 3 for one-slot programs, see dvm_vm_kernel).
// TWO: the build for launches that are known to run with two tile slots: the one-slot path is compiled out (the
// tile loop is short enough that every branch in it shows: +1.6 % on C2).
// DENSE: the build for programs whose loads are all one thread's (dense tiles and row vectors: no row-by-row copies, no
// per-row scalar inputs, no outer dims to decompose): those paths are compiled out of the load issue and of the
// operand addressing (+5 % on C2).
// AL: the build for programs all of whose operands are aligned like the tile's chunks (16-byte aligned tensors, rows a
// whole number of 16-byte units): the realignment of reads and the row shift are compiled out (+3 % on C2).
// FULL: the build for programs whose rows all fill the tile's slots exactly (columns = threads per row x elements per
// thread, one column block, no shorter last row): a thread's slots are all valid or -- past the last row -- all
// empty, so the slot masks, the sanitising of reductions and the element-wise store path are compiled out (+3 % on C2).
template <int V, int PW, bool SINGLE, bool HEAVY, bool PHASED = false, int CTAS = DVM_LEAN_MIN_CTAS, bool TWO = false, bool DENSE = false,
          bool AL = false, bool FULL = false>
__global__ void __launch_bounds__(THREADS, CTAS) dvm_vm_lean_kernel(const __grid_constant__ VMParams<PW> prm) {
  constexpr uint32_t kSingleProg = 3;  // directory of a one-program launch: [offset][0][n_tiles]
  constexpr int VP = V / 2;            // float2 pairs per tile register
  constexpr int NG = V / 8;            // 8-slot groups of a tile register
  constexpr uint32_t PSTRIDE = THREADS * 16;
  extern __shared__ __align__(16) uint32_t s_dyn[];
  __shared__ float s_red[2][THREADS / 32];
  __shared__ uint32_t s_next[2];
  __shared__ float s_S[DVM_MAX_SREGS][THREADS];
  __shared__ __align__(8) unsigned long long s_bar[2];
  __shared__ volatile uint32_t s_abort;

  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const uint32_t local_base = static_cast<uint32_t>(__cvta_generic_to_shared(s_dyn)) + DVM_LOCAL_UNIT;
  const uint32_t bar0 = static_cast<uint32_t>(__cvta_generic_to_shared(s_bar));
  const uint32_t n_prog = SINGLE ? 1u : prm.n_programs;
  const bool use_queue = SINGLE ? false : prm.use_queue != 0;
  // one tile slot (DVM_F_ONE_SLOT, one-program launches): both slots are the same memory, a tile's loads start
  // when the previous tile is done; the SM's other CTA computes meanwhile
  // (the builds for three resident CTAs only ever run one-slot launches: there the two-slot path folds away)
  const bool one_slot = TWO ? false : (SINGLE && (CTAS == 3 || prm.levels == 2));
#define CW(i) (prm.words[(i)])

  if (tid == 0) {
    s_abort = 0;
    vm_mbar_init(bar0, THREADS);
    vm_mbar_init(bar0 + 8, THREADS);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // ---- the rows of a tile, as far as this thread is concerned ----
  struct Rows {
    uint32_t row, col0;    // this thread's row of the dominant shape (may lie past the end), first column of the block
    int ncols;             // valid columns of that row inside the column block (0: nothing to do)
    uint32_t phase;        // phased programs: the tile's phase, and whether its column block is the row's last
    bool last_block;
  };
  struct Coord { uint32_t i0, i1, i2; };  // a row's coordinates over the collapsed outer dims
  auto tile_rows = [&](uint32_t prog, uint32_t local_tile, int as_tid) -> Rows {
    Rows r;
    const uint32_t geom = CW(prog + DVM_H_GEOM);
    const int lgG = geom & 0xff;
    const uint32_t CB = CW(prog + DVM_H_COL_BLOCKS);
    uint32_t rb = local_tile, cb = 0;
    if (CB > 1) { rb = local_tile / CB; cb = local_tile - rb * CB; }
    if constexpr (PHASED) {  // tile -> (row, phase, column block): the row's tiles are consecutive, phase by phase
      rb = local_tile / prm.row_tiles;
      const uint32_t sub = local_tile - rb * prm.row_tiles;
      r.phase = sub / CB;
      cb = sub - r.phase * CB;
      r.last_block = cb == CB - 1;
    }
    const uint32_t rows = CW(prog + DVM_H_ROWS_LO);
    r.row = rb * (uint32_t)(THREADS >> lgG) + (uint32_t)(as_tid >> lgG);
    const uint32_t ctile = CW(prog + DVM_H_COL_TILE);
    r.col0 = cb * ctile;
    const uint32_t cend = (r.row == rows - 1) ? CW(prog + DVM_H_LAST_ROW_COLS) : CW(prog + DVM_H_COLS);
    r.ncols = (r.row < rows && cend > r.col0) ? (int)min(cend - r.col0, ctile) : 0;
    return r;
  };
  auto coords = [&](uint32_t prog, uint32_t row) -> Coord {
    Coord c;
    c.i0 = row;
    c.i1 = c.i2 = 0;
    if (!DENSE && ((CW(prog + DVM_H_GEOM) >> 24) & DVM_F_OUTER_DIMS)) {
      // row -> coordinates over the outer dims: two divisions by multiply-and-shift (the linker left the
      // multipliers where the kernel type, code size, tile count and total words were)
      const uint32_t n0 = CW(prog + DVM_H_OUTER0), n1 = CW(prog + DVM_H_OUTER1);
      const uint32_t q = vm_magic_div(row, CW(prog + DVM_H_KERNEL_TYPE), CW(prog + DVM_H_CODE_WORDS));
      c.i0 = row - q * n0;
      c.i2 = vm_magic_div(q, CW(prog + DVM_H_N_TILES), CW(prog + DVM_H_TOTAL_WORDS));
      c.i1 = q - c.i2 * n1;
    }
    return c;
  };
  // element offset of the row (plus the column block start, for operands that have columns) inside operand d
  auto row_offset = [&](uint32_t prog, uint32_t d, const Rows& r) -> unsigned long long {
    const Coord c = coords(prog, r.row);
    unsigned long long off = (unsigned long long)c.i0 * CW(d + DVM_OPD_STRIDE0);
    off += (unsigned long long)c.i1 * CW(d + DVM_OPD_STRIDE1) + (unsigned long long)c.i2 * CW(d + DVM_OPD_STRIDE2);
    if ((CW(d + DVM_OPD_INFO) >> 16) & 0xff) off += r.col0;
    return off;
  };
  auto row_offset32 = [&](uint32_t prog, uint32_t d, const Rows& r) -> uint32_t {  // low bits: all an address phase needs
    const Coord c = coords(prog, r.row);
    uint32_t off = c.i0 * CW(d + DVM_OPD_STRIDE0) + c.i1 * CW(d + DVM_OPD_STRIDE1) + c.i2 * CW(d + DVM_OPD_STRIDE2);
    if ((CW(d + DVM_OPD_INFO) >> 16) & 0xff) off += r.col0;
    return off;
  };
  auto tensor_ptr = [&](uint32_t prog, uint32_t d) -> unsigned long long {
    const uint32_t tp = prog + DVM_HDR_WORDS + 2 * (CW(d + DVM_OPD_INFO) & 0xff);
    return (unsigned long long)CW(tp) | ((unsigned long long)CW(tp + 1) << 32);
  };
  auto opd_base = [&](uint32_t prog) -> uint32_t { return prog + DVM_HDR_WORDS + 2 * (CW(prog + DVM_H_COUNTS) & 0xff); };
  auto lreg_base = [&](uint32_t prog) -> uint32_t { return opd_base(prog) + ((CW(prog + DVM_H_COUNTS) >> 16) & 0xff) * DVM_OPD_WORDS; };
  auto body_base = [&](uint32_t prog) -> uint32_t { return lreg_base(prog) + ((CW(prog + DVM_H_GEOM) >> 16) & 0xff); };
  auto slot_base = [&](int slot) -> uint32_t { return local_base + (slot ? prm.slot_bytes : 0u); };

  // ---- load section of a tile: bulk copies into the images of slot `slot`; every thread arrives once ----
  auto issue_loads = [&](uint32_t prog, uint32_t local_tile, int slot, bool first_of_program) {
    const uint32_t bar = bar0 + 8 * slot;
    const uint32_t geom = CW(prog + DVM_H_GEOM);
    const int lgG = geom & 0xff;
    const int t = tid & ((1 << lgG) - 1);
    const bool by_row = DENSE ? false : ((geom >> 24) & DVM_F_LOADS_BY_ROW) != 0;
    const bool scalars = DENSE ? false : ((CW(prog + DVM_H_LOCAL) >> 16) & 0xff) != 0;
    const uint32_t load_words = CW(prog + DVM_H_LOAD_WORDS);
    // A program whose copies are all thread 0's (dense tiles, row vectors): the lanes of warp 0 take one load
    // instruction each, as thread 0 would -- the warp walks the load section once, not once per instruction.
    const bool by_lane = !scalars && !by_row;
    if (by_lane ? (warp == 0 && (uint32_t)lane < load_words) : (tid == 0 || scalars || (by_row && t == 0))) {
      const int me = by_lane ? 0 : tid;  // (the thread whose part of the tile this thread copies)
      const Rows r = tile_rows(prog, local_tile, me);
      const uint32_t opd0 = opd_base(prog), lreg0 = lreg_base(prog), body0 = body_base(prog);
      const uint32_t sb = slot_base(slot);
      const int Vv = V;
      for (uint32_t pc = by_lane ? (uint32_t)lane : 0u; pc < (by_lane ? (uint32_t)lane + 1u : load_words); ++pc) {
        const uint32_t w0 = CW(body0 + pc);
        const uint32_t d = opd0 + DVM_INSN_B(w0) * DVM_OPD_WORDS;
        const uint32_t lg_es = ((CW(d + DVM_OPD_INFO) >> 8) & 0xff) == DVM_DT_BF16 ? 1 : 2;
        if (DVM_INSN_OP(w0) == DVM_OP_LDG) {
          const uint32_t lw = CW(lreg0 + (DVM_INSN_A(w0) & 0x7f));
          const uint32_t mode = (lw >> 16) & 0xf;
          uint32_t dst = sb + (lw & 0xffffu) * DVM_LOCAL_UNIT;
          unsigned long long a = 0, n_el = 0;
          bool mine = false;
          if (mode == DVM_LM_BLOCK) {
            if (me == 0) {  // thread 0's row is the tile's first: the whole tile is one byte range from there
              mine = true;
              const uint32_t rows = CW(prog + DVM_H_ROWS_LO), C = CW(prog + DVM_H_COLS);
              const uint32_t rv = min((uint32_t)(THREADS >> lgG), rows - r.row);
              const uint32_t last = (r.row + rv == rows) ? CW(prog + DVM_H_LAST_ROW_COLS) : C;
              a = (unsigned long long)r.row * C;
              n_el = (unsigned long long)(rv - 1) * C + last;
            }
          } else if (!DENSE && mode == DVM_LM_ROWS) {
            if (t == 0 && r.ncols > 0) {
              mine = true;
              a = row_offset(prog, d, r);
              n_el = (unsigned long long)r.ncols;
              dst += (uint32_t)(tid >> lgG) * DVM_ROW_PITCH(1 << lgG, Vv, 1u << lg_es);
            }
          } else {  // a row vector: the same for every tile (BCAST: loaded once per slot and program) or column block
            if ((first_of_program || mode == DVM_LM_BCAST_TILE) && me == 0) {
              mine = true;
              a = r.col0;
              n_el = min(CW(prog + DVM_H_COLS) - r.col0, CW(prog + DVM_H_COL_TILE));
            }
          }
          if (mine) {
            const unsigned long long g0 = tensor_ptr(prog, d) + (a << lg_es);
            const unsigned long long gs = g0 & ~15ull, ge = (g0 + (n_el << lg_es) + 15ull) & ~15ull;
            const uint32_t bytes = (uint32_t)(ge - gs);
            asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
            vm_bulk_load(dst, reinterpret_cast<const void*>(gs), bytes, bar);
          }
        } else {  // DVM_OP_LDS: one value per row into this thread's scalar slot
          const char* p = reinterpret_cast<const char*>(tensor_ptr(prog, d) + (row_offset(prog, d, r) << lg_es));
          const uint32_t w = (uint32_t)DVM_INSN_A(w0);
          const uint32_t dst = sb + (CW(prog + DVM_H_LOCAL2) & 0xffffu) * DVM_LOCAL_UNIT + (uint32_t)tid * 16 + (w >> 2) * PSTRIDE + (w & 3) * 4;
          if (r.ncols > 0) {
            if (lg_es == 1) {
              const float v = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(p));
              asm volatile("st.shared.f32 [%0], %1;" ::"r"(dst), "f"(v) : "memory");
            } else {
              cp_async4(dst, p);
            }
          }
        }
      }
    }
    vm_mbar_arrive(bar);
  };

  float2 A[VP];
#pragma unroll
  for (int i = 0; i < VP; ++i) A[i] = make_float2(0.f, 0.f);
#define DVM_EACH_PAIR _Pragma("unroll") for (int i = DVM_P0; i < DVM_P1; ++i)
#define DVM_P0 0
#define DVM_P1 VP
  // ACC = ACC op Y, eight operations (Y: an expression of i)
#define DVM_ARITH(SUB, YX, YY)                                                                                         \
  switch (SUB) {                                                                                                       \
    case DVM_A_ADD: DVM_EACH_PAIR A[i] = __fadd2_rn(A[i], make_float2(YX, YY)); break;                                 \
    case DVM_A_SUB: DVM_EACH_PAIR A[i] = __ffma2_rn(make_float2(YX, YY), make_float2(-1.f, -1.f), A[i]); break;        \
    case DVM_A_RSUB: DVM_EACH_PAIR A[i] = __ffma2_rn(A[i], make_float2(-1.f, -1.f), make_float2(YX, YY)); break;       \
    case DVM_A_MUL: DVM_EACH_PAIR A[i] = __fmul2_rn(A[i], make_float2(YX, YY)); break;                                 \
    case DVM_A_DIV: DVM_EACH_PAIR A[i] = make_float2(fast_div(A[i].x, YX), fast_div(A[i].y, YY)); break;               \
    case DVM_A_RDIV: DVM_EACH_PAIR A[i] = make_float2(fast_div(YX, A[i].x), fast_div(YY, A[i].y)); break;              \
    case DVM_A_MIN: DVM_EACH_PAIR A[i] = make_float2(A[i].x < (YX) ? A[i].x : (YX), A[i].y < (YY) ? A[i].y : (YY)); break; \
    default: DVM_EACH_PAIR A[i] = make_float2(A[i].x > (YX) ? A[i].x : (YX), A[i].y > (YY) ? A[i].y : (YY)); break;    \
  }

  uint32_t prog_idx = 0;
  uint32_t tile = blockIdx.x + (SINGLE ? prm.tile_begin : 0u);
  if constexpr (PHASED) tile = blockIdx.x * prm.row_tiles;
  uint32_t iter = 0;
  int red_par = 0;
  int buf = 0;
  unsigned err = 0;
  uint32_t slot_prog[2] = {0xffffffffu, 0xffffffffu};

  // validity of this thread's slots: slot s < 8 is valid iff bit s of hm, slot s >= 8 iff s < nvalid
  // (kept from tile to tile while program, row length and shift stay the same)
  uint32_t m_prog = 0xffffffffu;
  int m_ncols = -1, m_shift = -1;
  uint32_t hm = 0, fullmask = 0, partmask = 0;
  int nvalid = 0;
  bool all_valid = false;

  if (tile < prm.total_tiles && !one_slot) {
    if (!SINGLE) while (prog_idx + 1 < n_prog && tile >= CW(n_prog + prog_idx + 1)) ++prog_idx;
    issue_loads(SINGLE ? kSingleProg : CW(prog_idx), SINGLE ? tile : tile - CW(n_prog + prog_idx), 0, true);
    slot_prog[0] = prog_idx;
    cp_async_commit();
  }

  while (tile < prm.total_tiles) {
    // ---- Algorithm 2, outer loop ----
    if (use_queue && tid == 0) s_next[iter & 1] = atomicAdd(&prm.queue[0], 1u) + gridDim.x;
    __syncthreads();  // everybody is done with the previous tile: its slot may be refilled
    if (s_abort) break;
    uint32_t next = use_queue ? s_next[iter & 1] : tile + gridDim.x;
    if constexpr (PHASED) {  // the next tile of this row, or the first tile of this CTA's next row
      next = tile + 1;
      if (next % prm.row_tiles == 0) next += (gridDim.x - 1) * prm.row_tiles;
    }
    ++iter;
    uint32_t next_prog_idx = prog_idx;
    if (SINGLE && one_slot) {
      // this tile's own loads, now that nobody reads the slot any more (the first tile also brings the row vectors)
      issue_loads(kSingleProg, tile, 0, iter == 1);
      cp_async_commit();
      cp_async_wait<0>();
      if (!vm_mbar_wait(bar0, (iter - 1) & 1)) {
        err = ST_TIMEOUT;
        s_abort = 1;
      }
    } else {
      if (next < prm.total_tiles) {
        if (!SINGLE) while (next_prog_idx + 1 < n_prog && next >= CW(n_prog + next_prog_idx + 1)) ++next_prog_idx;
        const bool first = buf ? slot_prog[0] != next_prog_idx : slot_prog[1] != next_prog_idx;
        issue_loads(SINGLE ? kSingleProg : CW(next_prog_idx), SINGLE ? next : next - CW(n_prog + next_prog_idx), buf ^ 1, first);
        if (buf) slot_prog[0] = next_prog_idx; else slot_prog[1] = next_prog_idx;
        cp_async_commit();
        cp_async_wait<1>();
      } else {
        cp_async_wait<0>();
      }
      if (!vm_mbar_wait(bar0 + 8 * buf, ((iter - 1) >> 1) & 1)) {
        err = ST_TIMEOUT;
        s_abort = 1;
      }
    }

    // ---- this tile: rows, shift, slot masks, where this thread's chunks lie ----
    const uint32_t prog = SINGLE ? kSingleProg : CW(prog_idx);
    const Rows r = tile_rows(prog, SINGLE ? tile : tile - CW(n_prog + prog_idx), tid);
    const uint32_t geom = CW(prog + DVM_H_GEOM);
    const int lgG = geom & 0xff;
    const int lgW = ((geom >> 8) & 0xff) == 8 ? 3 : 2;
    const uint32_t flags = geom >> 24;
    const int G = 1 << lgG;
    const int t = tid & (G - 1);
    const uint32_t rr = (uint32_t)(tid >> lgG);
    const uint32_t C = CW(prog + DVM_H_COLS);
    const uint32_t sb = slot_base(buf);
    int shift = 0;
    if (!AL && !(flags & DVM_F_ALIGNED)) {
      const uint32_t d = opd_base(prog) + CW(prog + DVM_H_PRIMARY) * DVM_OPD_WORDS;
      const uint32_t lg_es = ((CW(d + DVM_OPD_INFO) >> 8) & 0xff) == DVM_DT_BF16 ? 1 : 2;
      const uint32_t base_el = (uint32_t)tensor_ptr(prog, d) >> lg_es;
      const uint32_t off = (flags & DVM_F_PRIMARY_DENSE) ? r.row * C + r.col0 : row_offset32(prog, d, r);
      shift = (int)((base_el + off) & (uint32_t)((1 << lgW) - 1));
    }
    const int cbase = (t << lgW) - shift;
    const uint32_t img = rr * C + (uint32_t)cbase;   // element offset of this thread's first chunk in a dense tile image
    const uint32_t row0C = (r.row - rr) * C;         // element offset of the tile's first row in a dense tensor (low bits)
    // (the test is made warp-wide: the vote below needs every lane)
    if constexpr (FULL) {
      const int nch = V >> lgW;
      const bool ok = r.ncols > 0;
      nvalid = ok ? V : 0;
      hm = ok ? 0xffu : 0u;
      partmask = 0u;
      fullmask = ok ? ((nch >= 32) ? 0xffffffffu : ((1u << nch) - 1u)) : 0u;
      all_valid = true;  // (a row past the end reduces whatever its slots hold: nobody reads the result)
    } else if (__any_sync(0xffffffffu, m_prog != prog || m_ncols != r.ncols || m_shift != shift)) {
      m_prog = prog; m_ncols = r.ncols; m_shift = shift;
      // In mapping coordinates the row segment is [shift, shift + ncols); this thread owns chunks t, t + G, ...
      const int W = 1 << lgW;
      const int nch = V >> lgW;
      const int n2 = r.ncols > 0 ? r.ncols + shift : 0;
      const int avail = (n2 >> lgW) - t;
      int nf = avail > 0 ? ((avail + G - 1) >> lgG) : 0;
      nf = nf < nch ? nf : nch;
      int rem = nf < nch ? n2 - ((t + (nf << lgG)) << lgW) : 0;
      rem = rem > 0 ? (rem < W ? rem : W) : 0;
      nvalid = (nf << lgW) + rem;
      fullmask = (nf >= 32) ? 0xffffffffu : ((1u << nf) - 1u);
      partmask = rem > 0 ? (1u << nf) : 0u;
      hm = nvalid >= 8 ? 0xffu : ((1u << nvalid) - 1u);
      if (shift > 0 && t == 0 && r.ncols > 0) {  // head chunk of a misaligned row: slots [0, shift) lie before it
        hm &= ~((1u << shift) - 1u);
        fullmask &= ~1u;
        partmask |= 1u;
      }
      all_valid = __all_sync(0xffffffffu, nvalid == V && hm == 0xffu);
    }

    // Byte address of this thread's first chunk of the local register an operand word names (its low four bits:
    // the operand's misalignment against the tile's chunks).
    auto opw_addr = [&](uint32_t ow) -> uint32_t {
      const uint32_t mode = (ow >> 18) & 7u;
      const uint32_t lg_es = 1u + ((ow >> 21) & 1u);
      const uint32_t base_lo = (ow >> 22) & 15u;
      uint32_t a = sb + (ow & 0x3ffffu);
      if (mode == DVM_LM_BLOCK) return a + (img << lg_es) + ((base_lo + (row0C << lg_es)) & 15u);
      uint32_t off;
      if (!DENSE && mode == DVM_LM_ROWS) {
        off = row_offset32(prog, opd_base(prog) + (ow >> 26) * DVM_OPD_WORDS, r);
        a += rr * (((uint32_t)V << (lgG + lg_es)) + 32u);
      } else {
        off = r.col0;
      }
      return a + ((base_lo + (off << lg_es)) & 15u) + ((uint32_t)cbase << lg_es);
    };
    // Slots outside the row get the identity of the reduction that follows.  Only the 8-slot groups the row's
    // head or tail cuts are touched (at most two per thread); groups wholly outside are skipped by the reduction.
    auto sanitize = [&](float ident) {
      if (hm != 0xffu && hm != 0u) {
#pragma unroll
        for (int e = 0; e < 8; ++e)
          if (!((hm >> e) & 1u)) { if (e & 1) A[e >> 1].y = ident; else A[e >> 1].x = ident; }
      }
      if (NG > 1 && nvalid > 8 && (nvalid & 7)) {
        const int g = nvalid >> 3, keep = nvalid & 7;
#pragma unroll
        for (int gg = 1; gg < NG; ++gg)
          if (gg == g) {
#pragma unroll
            for (int e = 0; e < 8; ++e)
              if (e >= keep) { if (e & 1) A[4 * gg + (e >> 1)].y = ident; else A[4 * gg + (e >> 1)].x = ident; }
          }
      }
    };
    auto group_on = [&](int g) -> bool { return g == 0 ? hm != 0u : nvalid > 8 * g; };

    // ---- Algorithm 2, inner loop: the linked compute section, one record per step ----
    uint32_t rp = prog + CW(prog + DVM_H_MAGIC);  // (the launch put the records' offset where the magic word was)
    bool stop = false;  // (phased programs: a phase marker ended this tile's walk)
    for (;;) {
      const uint4 rec = *reinterpret_cast<const uint4*>(&CW(rp));
      rp += 4;
      const uint32_t h = rec.x & 0xffu;
      const uint32_t sub = (rec.x >> 8) & 0xffu;
      const uint32_t ra = (rec.x >> 16) & 0xffu;
      if (h == DVM_LK_END) break;
      // two dispatch levels: the records of the bf16 sweeps (load, multiply-add, exponential, reduction, store) first
      if (h <= DVM_LK_HOT_LAST) {
      switch (h) {
        case DVM_LK_LDA_BF16: {
          uint32_t R[V / 2];
          lean_raw_bf16<V, AL>(R, opw_addr(lean_opaque<1>(rec.y)), (uint32_t)(G << 4));
          DVM_EACH_PAIR A[i] = lean_widen(R[i]);
        } break;
        case DVM_LK_LD2_BF16: {  // ACC = L[x] op L[y] (* imm): add / sub / rsub / mul
          uint32_t R[V / 2];
          lean_raw_bf16<V, AL>(R, opw_addr(lean_opaque<2>(rec.y)), (uint32_t)(G << 4));
          DVM_EACH_PAIR A[i] = lean_widen(R[i]);
          lean_raw_bf16<V, AL>(R, opw_addr(lean_opaque<42>(rec.z)), (uint32_t)(G << 4));
          if (sub == DVM_A_ADD) { DVM_EACH_PAIR A[i] = __fadd2_rn(A[i], lean_widen(R[i])); }
          else if (sub == DVM_A_MUL) { DVM_EACH_PAIR A[i] = __fmul2_rn(A[i], lean_widen(R[i])); }
          else if (sub == DVM_A_SUB) { DVM_EACH_PAIR A[i] = __ffma2_rn(lean_widen(R[i]), make_float2(-1.f, -1.f), A[i]); }
          else { DVM_EACH_PAIR A[i] = __ffma2_rn(A[i], make_float2(-1.f, -1.f), lean_widen(R[i])); }
          if (rec.x >> 24) {
            const float m = __uint_as_float(rec.w);
            DVM_EACH_PAIR A[i] = __fmul2_rn(A[i], make_float2(m, m));
          }
        } break;
        case DVM_LK_BIN_BF16: {
          uint32_t R[V / 2];
          lean_raw_bf16<V, AL>(R, opw_addr(lean_opaque<3>(rec.y)), (uint32_t)(G << 4));
          if (rec.x >> 24) {  // ACC = ACC * S[.] * L[y]
            const float m = s_S[(rec.x >> 24) - 1][tid];
            DVM_EACH_PAIR A[i] = __fmul2_rn(__fmul2_rn(A[i], make_float2(m, m)), lean_widen(R[i]));
          } else {
            DVM_ARITH(sub, __uint_as_float(R[i] << 16), __uint_as_float(R[i] & 0xffff0000u))
          }
        } break;
        case DVM_LK_FMA: {  // ACC = ACC * m + c, m and c immediates or per-row scalars: add / sub / rsub / mul / div by a scalar
          const uint32_t ra_ = lean_opaque<9>(ra);
          float m = (sub & 1u) ? s_S[ra_][tid] : __uint_as_float(rec.y);
          float c = (sub & 2u) ? s_S[rec.x >> 24][tid] : __uint_as_float(rec.z);
          if (sub & 4u) m = fast_rcp(m);
          if (sub & 8u) c = -c;
          DVM_EACH_PAIR A[i] = __ffma2_rn(A[i], make_float2(m, m), make_float2(c, c));
        } break;
        case DVM_LK_EXPS: {
          const float m = -s_S[lean_opaque<11>(ra)][tid];
          if (sub) {  // every output of the program is bf16: the one-piece exponential
            const float nc = m * 1.44269502162933349609375f;
            DVM_EACH_PAIR A[i] = lean_exp2_fast(A[i], nc);
          } else {
            DVM_EACH_PAIR A[i] = lean_exp2(__fadd2_rn(A[i], make_float2(m, m)));
          }
        } break;
        case DVM_LK_RED: {
          // ---- row reduction (Table 1, Sum / Max / Min with N = 1) ----
          const int rop = (int)sub;
          bool accumulate = false, finish = true;
          if constexpr (PHASED) {
            const uint32_t tag = rec.x >> 28;
            if (tag) {  // the reduction belongs to one phase: it runs over that phase's blocks and completes in the last
              if (tag - 1 != r.phase) break;
              accumulate = r.col0 != 0;
              finish = r.last_block;
            }
          }
          const bool is_sum = rop == DVM_R_SUM || rop == DVM_R_SUMSQ;
          const float ident = is_sum ? 0.f : (rop == DVM_R_MAX ? -INFINITY : INFINITY);
          if (!all_valid) sanitize(ident);
          float v;
          if (is_sum) {
            // four partial sums per thread, one per pair of an 8-slot group (independent chains), then a tree
            float2 acc[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[q] = make_float2(0.f, 0.f);
#pragma unroll
            for (int g = 0; g < NG; ++g)
              if (all_valid || group_on(g)) {
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[q] = rop == DVM_R_SUM ? __fadd2_rn(acc[q], A[4 * g + q]) : __ffma2_rn(A[4 * g + q], A[4 * g + q], acc[q]);
              }
            const float2 a2 = __fadd2_rn(__fadd2_rn(acc[0], acc[1]), __fadd2_rn(acc[2], acc[3]));
            v = a2.x + a2.y;
#pragma unroll
            for (int sh = 1; sh < 32; sh <<= 1)
              if (sh < G) v += __shfl_xor_sync(0xffffffffu, v, sh);
          } else {
            const bool mx = rop == DVM_R_MAX;
            float m4[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) m4[q] = ident;
#pragma unroll
            for (int g = 0; g < NG; ++g)
              if (all_valid || group_on(g)) {
#pragma unroll
                for (int q = 0; q < 4; ++q) m4[q] = mx ? fmaxf(m4[q], fmaxf(A[4 * g + q].x, A[4 * g + q].y)) : fminf(m4[q], fminf(A[4 * g + q].x, A[4 * g + q].y));
              }
            v = mx ? fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) : fminf(fminf(m4[0], m4[1]), fminf(m4[2], m4[3]));
            if (G >= 32) {  // the whole warp holds one row: the warp-wide fp32 max / min instruction of sm_100a
              float w;
              if (mx) asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(w) : "f"(v));
              else asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(w) : "f"(v));
              v = w;
            } else {
#pragma unroll
              for (int sh = 1; sh < 32; sh <<= 1)
                if (sh < G) {
                  const float x = __shfl_xor_sync(0xffffffffu, v, sh);
                  v = mx ? fmaxf(v, x) : fminf(v, x);
                }
            }
          }
          if (G > 32) {
            if (lane == 0) s_red[red_par][warp] = v;
            const int wpg = G >> 5;  // warps per row group: 2, 4 or 8
            if (wpg == 8) __syncthreads();
            else asm volatile("bar.sync %0, %1;" ::"r"(1 + (warp >> (lgG - 5))), "r"(G) : "memory");
            const float* pr = &s_red[red_par][warp & ~(wpg - 1)];
            float x[8];
            x[0] = pr[0]; x[1] = pr[1];
#pragma unroll
            for (int i = 2; i < 8; ++i) x[i] = ident;
            if (wpg > 2) { x[2] = pr[2]; x[3] = pr[3]; }
            if (wpg > 4) { x[4] = pr[4]; x[5] = pr[5]; x[6] = pr[6]; x[7] = pr[7]; }
            if (rop == DVM_R_MAX) v = fmaxf(fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3])), fmaxf(fmaxf(x[4], x[5]), fmaxf(x[6], x[7])));
            else if (rop == DVM_R_MIN) v = fminf(fminf(fminf(x[0], x[1]), fminf(x[2], x[3])), fminf(fminf(x[4], x[5]), fminf(x[6], x[7])));
            else v = ((x[0] + x[1]) + (x[2] + x[3])) + ((x[4] + x[5]) + (x[6] + x[7]));
            red_par ^= 1;
          }
          if constexpr (PHASED) {
            if (accumulate) {
              const float prev = s_S[ra][tid];
              v = rop == DVM_R_MAX ? fmaxf(prev, v) : (rop == DVM_R_MIN ? fminf(prev, v) : prev + v);
            }
          }
          if (PHASED ? (((rec.x >> 24) & 1u) != 0 && finish) : (rec.x >> 24) != 0) {  // the scalar multiply-add(-unary) that followed the reduction, rounded like the separate steps
            v = __fadd_rn(__fmul_rn(v, __uint_as_float(rec.z)), __uint_as_float(rec.w));
            if (rec.y != 0xffu) v = scalar_unary((int)rec.y, v);
          }
          s_S[lean_opaque<13>(ra)][tid] = v;
        } break;
        case DVM_LK_STG: {
          if constexpr (PHASED) {
            if ((rec.x >> 24) && (rec.x >> 24) - 1 != r.phase) break;  // a phased program stores in its last phase
          }
          const int lg_es = (int)lean_opaque<54>(ra);
          const unsigned long long base = (unsigned long long)lean_opaque<14>(rec.y) | ((unsigned long long)rec.z << 32);
          const unsigned long long el0 = (unsigned long long)r.row * C + r.col0;
          char* p = reinterpret_cast<char*>(base + (el0 << lg_es));
          char* q0 = p + ((long long)cbase << lg_es);
          const long long qstep = (long long)((G << lgW) << lg_es);
          const bool al = (reinterpret_cast<uintptr_t>(q0) & 15) == 0;
          const uint32_t fast = al ? fullmask : 0u;
          const uint32_t slow = partmask | (fullmask & ~fast);
          if (lg_es == 1) {  // bf16: chunks of 8, chunk j = group j
#pragma unroll
            for (int j = 0; j < V / 8; ++j)
              if ((fast >> j) & 1) {
                uint32_t pk[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  const __nv_bfloat162 b = __floats2bfloat162_rn(A[4 * j + q].x, A[4 * j + q].y);
                  pk[q] = *reinterpret_cast<const uint32_t*>(&b);
                }
                *reinterpret_cast<uint4*>(q0 + j * qstep) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
              }
          } else if (lgW == 3) {
#pragma unroll
            for (int j = 0; j < V / 8; ++j)
              if ((fast >> j) & 1) {
                *reinterpret_cast<float4*>(q0 + j * qstep) = make_float4(A[4 * j].x, A[4 * j].y, A[4 * j + 1].x, A[4 * j + 1].y);
                *reinterpret_cast<float4*>(q0 + j * qstep + 16) = make_float4(A[4 * j + 2].x, A[4 * j + 2].y, A[4 * j + 3].x, A[4 * j + 3].y);
              }
          } else {
#pragma unroll
            for (int j = 0; j < V / 4; ++j)
              if ((fast >> j) & 1)
                *reinterpret_cast<float4*>(q0 + j * qstep) = make_float4(A[2 * j].x, A[2 * j].y, A[2 * j + 1].x, A[2 * j + 1].y);
          }
          if (slow) {
            // chunks cut by the row's head or tail (or stored at another alignment than the tile's chunks):
            // element stores, one 8-slot group at a time.  (The column arithmetic hangs on an opaque copy of the
            // chunk base: it is the same for every record of a tile, and the compiler would otherwise compute all
            // of it at the top of every tile, for a path few threads take.)
            const int cb = (int)lean_opaque<90>((uint32_t)cbase);
#pragma unroll
            for (int g = 0; g < NG; ++g) {
              const uint32_t gm = lgW == 3 ? ((slow >> g) & 1u) : ((slow >> (2 * g)) & 3u);
              if (gm) {
                // first column of the group's first (and, with chunks of 4, second) chunk
                const int c0 = cb + ((lgW == 3 ? g : 2 * g) << (lgG + lgW));
                const int c1 = lgW == 3 ? c0 + 4 : c0 + (1 << (lgG + 2));
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  const int col = e < 4 ? c0 + e : c1 + (e - 4);
                  const bool in_slow = lgW == 3 ? true : ((gm >> (e >> 2)) & 1u) != 0;
                  const float val = (e & 1) ? A[4 * g + (e >> 1)].y : A[4 * g + (e >> 1)].x;
                  if (in_slow && col >= 0 && col < r.ncols) {
                    if (lg_es == 1) *reinterpret_cast<__nv_bfloat16*>(p + (long long)col * 2) = __float2bfloat16_rn(val);
                    else *reinterpret_cast<float*>(p + (long long)col * 4) = val;
                  }
                }
              }
            }
          }
        } break;
        default: break;
      }
      } else {
      switch (h) {
        case DVM_LK_LDA_F32: {  // (in two halves: the raw words of a whole fp32 tile register would crowd the registers)
          const uint32_t a = opw_addr(lean_opaque<4>(rec.y));
#define DVM_LDA_F32_HALF(H)                                                                               \
          {                                                                                               \
            uint32_t R[V / 2];                                                                            \
            if (lgW == 3) lean_raw_f32<2, (H) * (V / 16), ((H) + 1) * (V / 16), AL>(R, a, (uint32_t)(G << 5)); \
            else lean_raw_f32<1, (H) * (V / 8), ((H) + 1) * (V / 8), AL>(R, a, (uint32_t)(G << 4));            \
            _Pragma("unroll") for (int i = 0; i < VP / 2; ++i)                                            \
              A[(H) * (VP / 2) + i] = make_float2(__uint_as_float(R[2 * i]), __uint_as_float(R[2 * i + 1])); \
          }
          DVM_LDA_F32_HALF(0)
          DVM_LDA_F32_HALF(1)
#undef DVM_LDA_F32_HALF
        } break;
        case DVM_LK_BIN_F32: {
          const uint32_t a = opw_addr(lean_opaque<5>(rec.y));
          const bool pre = (rec.x >> 24) != 0;  // ACC = ACC * S[.] * L[y]
          const float m = pre ? s_S[(rec.x >> 24) - 1][tid] : 1.0f;
#define DVM_BIN_F32_HALF(H)                                                                               \
          {                                                                                               \
            uint32_t R[V / 2];                                                                            \
            if (lgW == 3) lean_raw_f32<2, (H) * (V / 16), ((H) + 1) * (V / 16), AL>(R, a, (uint32_t)(G << 5)); \
            else lean_raw_f32<1, (H) * (V / 8), ((H) + 1) * (V / 8), AL>(R, a, (uint32_t)(G << 4));            \
            if (pre) {                                                                                    \
              _Pragma("unroll") for (int i = (H) * (VP / 2); i < ((H) + 1) * (VP / 2); ++i)               \
                A[i] = __fmul2_rn(__fmul2_rn(A[i], make_float2(m, m)),                                    \
                                  make_float2(__uint_as_float(R[2 * i - (H) * (V / 2)]), __uint_as_float(R[2 * i + 1 - (H) * (V / 2)]))); \
            } else {                                                                                      \
              DVM_ARITH(sub, __uint_as_float(R[2 * i - (H) * (V / 2)]), __uint_as_float(R[2 * i + 1 - (H) * (V / 2)])) \
            }                                                                                             \
          }
#undef DVM_P0
#undef DVM_P1
#define DVM_P0 0
#define DVM_P1 (VP / 2)
          DVM_BIN_F32_HALF(0)
#undef DVM_P0
#undef DVM_P1
#define DVM_P0 (VP / 2)
#define DVM_P1 VP
          DVM_BIN_F32_HALF(1)
#undef DVM_P0
#undef DVM_P1
#define DVM_P0 0
#define DVM_P1 VP
#undef DVM_BIN_F32_HALF
        } break;
        case DVM_LK_LDA_PRIV: {
          const uint32_t a = sb + (lean_opaque<6>(rec.y) & 0x3ffffu) + (uint32_t)tid * 16;
#pragma unroll
          for (int q = 0; q < V / 4; ++q) {
            const uint4 v = lean_lds128(a + q * PSTRIDE);
            A[2 * q] = make_float2(__uint_as_float(v.x), __uint_as_float(v.y));
            A[2 * q + 1] = make_float2(__uint_as_float(v.z), __uint_as_float(v.w));
          }
        } break;
        case DVM_LK_BIN_PRIV: {
          const uint32_t a = sb + (lean_opaque<7>(rec.y) & 0x3ffffu) + (uint32_t)tid * 16;
          uint32_t R[V];
#pragma unroll
          for (int q = 0; q < V / 4; ++q) {
            const uint4 v = lean_lds128(a + q * PSTRIDE);
            R[4 * q] = v.x; R[4 * q + 1] = v.y; R[4 * q + 2] = v.z; R[4 * q + 3] = v.w;
          }
          DVM_ARITH(sub, __uint_as_float(R[2 * i]), __uint_as_float(R[2 * i + 1]))
        } break;
        case DVM_LK_BIN_ACC: {
          float2 Y[VP];
          DVM_EACH_PAIR Y[i] = A[i];
          DVM_ARITH(sub, Y[i].x, Y[i].y)
        } break;
        case DVM_LK_BINI:
        case DVM_LK_BINS: {  // (what the multiply-add form does not cover: rdiv, min, max)
          const uint32_t ra_ = lean_opaque<10>(ra);
          const float y = h == DVM_LK_BINS ? s_S[ra_][tid] : __uint_as_float(rec.y);
          if (sub == DVM_A_RDIV) { DVM_EACH_PAIR A[i] = make_float2(fast_div(y, A[i].x), fast_div(y, A[i].y)); }
          else if (sub == DVM_A_MIN) { DVM_EACH_PAIR A[i] = make_float2(A[i].x < y ? A[i].x : y, A[i].y < y ? A[i].y : y); }
          else { DVM_EACH_PAIR A[i] = make_float2(A[i].x > y ? A[i].x : y, A[i].y > y ? A[i].y : y); }
        } break;
        case DVM_LK_ACT: {
          if constexpr (HEAVY) {
            if (sub == DVM_ACT_GELU) { DVM_EACH_PAIR A[i] = packed_gelu(A[i]); }
            else { DVM_EACH_PAIR A[i] = packed_silu(A[i]); }
          } else {
            err = ST_BAD_CODE;
          }
        } break;
        case DVM_LK_UN: {
#define DVM_UN_CASE(U, EXPR)                                                          \
  case U:                                                                             \
    DVM_EACH_PAIR {                                                                   \
      float x = A[i].x; const float vx = (EXPR);                                      \
      x = A[i].y; const float vy = (EXPR);                                            \
      A[i] = make_float2(vx, vy);                                                     \
    }                                                                                 \
    break;
          switch (sub) {
            case DVM_U_EXP: DVM_EACH_PAIR A[i] = lean_exp2(A[i]); break;
            case DVM_U_EXP | 0x80: DVM_EACH_PAIR A[i] = lean_exp2_fast(A[i], 0.f); break;
            case DVM_U_SIGMOID | 0x80:
              DVM_EACH_PAIR {
                const float2 e = lean_exp2_fast(make_float2(-A[i].x, -A[i].y), 0.f);
                A[i] = make_float2(fast_rcp(1.0f + e.x), fast_rcp(1.0f + e.y));
              }
              break;
            DVM_UN_CASE(DVM_U_RSQRT, rsqrtf(x))
            DVM_UN_CASE(DVM_U_ABS, fabsf(x))
            case DVM_U_SIGMOID:
              DVM_EACH_PAIR {
                const float2 e = lean_exp2(make_float2(-A[i].x, -A[i].y));
                A[i] = make_float2(fast_rcp(1.0f + e.x), fast_rcp(1.0f + e.y));
              }
              break;
            DVM_UN_CASE(DVM_U_NEG, -x)
            DVM_UN_CASE(DVM_U_RECIP, fast_rcp(x))
            DVM_UN_CASE(DVM_U_RND_BF16, round_bf16(x))
            default:
              if constexpr (HEAVY) {
                switch (sub) {
                  DVM_UN_CASE(DVM_U_TRUNC_I32, trunc_i32(x))
                  DVM_UN_CASE(DVM_U_TRUNC_U8, trunc_u8(x))
                  DVM_UN_CASE(DVM_U_SQRT, sqrtf(x))
                  DVM_UN_CASE(DVM_U_LOG, logf(x))
                  case DVM_U_ERF: DVM_EACH_PAIR A[i] = packed_erf(A[i]); break;
                  DVM_UN_CASE(DVM_U_FLOOR, floorf(x))
                  DVM_UN_CASE(DVM_U_ROUND, rintf(x))
                  DVM_UN_CASE(DVM_U_TANH, tanhf(x))
                  default: err = ST_BAD_CODE; break;
                }
              } else {
                err = ST_BAD_CODE;
              }
              break;
          }
#undef DVM_UN_CASE
        } break;
        case DVM_LK_STGI: {  // Table 1, Cast: ACC stored as i32 (sub 1) or u8 (sub 2), converted toward zero
          if constexpr (PHASED) {
            if ((rec.x >> 24) && (rec.x >> 24) - 1 != r.phase) break;
          }
          const int lg_es = (int)lean_opaque<55>(ra);
          const unsigned long long base = (unsigned long long)lean_opaque<15>(rec.y) | ((unsigned long long)rec.z << 32);
          const unsigned long long el0 = (unsigned long long)r.row * C + r.col0;
          char* p = reinterpret_cast<char*>(base + (el0 << lg_es));
          char* q0 = p + ((long long)cbase << lg_es);
          const long long qstep = (long long)((G << lgW) << lg_es);
          // (a chunk of u8 is W bytes: its vector store wants that alignment; i32 goes in 16-byte vectors)
          const bool al = (reinterpret_cast<uintptr_t>(q0) & (lg_es == 0 ? (uintptr_t)((1 << lgW) - 1) : (uintptr_t)15)) == 0;
          const uint32_t fast = al ? fullmask : 0u;
          const uint32_t slow = partmask | (fullmask & ~fast);
          if (sub == 2) {  // Table 1, Cast: stored as u8, a chunk is W bytes
            if (lgW == 3) {
#pragma unroll
              for (int j = 0; j < V / 8; ++j)
                if ((fast >> j) & 1)
                  *reinterpret_cast<uint2*>(q0 + j * qstep) = make_uint2(pack_u8x4(A[4 * j].x, A[4 * j].y, A[4 * j + 1].x, A[4 * j + 1].y),
                                                                         pack_u8x4(A[4 * j + 2].x, A[4 * j + 2].y, A[4 * j + 3].x, A[4 * j + 3].y));
            } else {
#pragma unroll
              for (int j = 0; j < V / 4; ++j)
                if ((fast >> j) & 1)
                  *reinterpret_cast<uint32_t*>(q0 + j * qstep) = pack_u8x4(A[2 * j].x, A[2 * j].y, A[2 * j + 1].x, A[2 * j + 1].y);
            }
          } else {  // stored as i32
            if (lgW == 3) {
#pragma unroll
              for (int j = 0; j < V / 8; ++j)
                if ((fast >> j) & 1) {
                  *reinterpret_cast<uint4*>(q0 + j * qstep) = make_uint4(store_i32(A[4 * j].x), store_i32(A[4 * j].y), store_i32(A[4 * j + 1].x), store_i32(A[4 * j + 1].y));
                  *reinterpret_cast<uint4*>(q0 + j * qstep + 16) = make_uint4(store_i32(A[4 * j + 2].x), store_i32(A[4 * j + 2].y), store_i32(A[4 * j + 3].x), store_i32(A[4 * j + 3].y));
                }
            } else {
#pragma unroll
              for (int j = 0; j < V / 4; ++j)
                if ((fast >> j) & 1)
                  *reinterpret_cast<uint4*>(q0 + j * qstep) = make_uint4(store_i32(A[2 * j].x), store_i32(A[2 * j].y), store_i32(A[2 * j + 1].x), store_i32(A[2 * j + 1].y));
            }
          }
          if (slow) {
            const int cb = (int)lean_opaque<91>((uint32_t)cbase);
#pragma unroll
            for (int g = 0; g < NG; ++g) {
              const uint32_t gm = lgW == 3 ? ((slow >> g) & 1u) : ((slow >> (2 * g)) & 3u);
              if (gm) {
                const int c0 = cb + ((lgW == 3 ? g : 2 * g) << (lgG + lgW));
                const int c1 = lgW == 3 ? c0 + 4 : c0 + (1 << (lgG + 2));
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  const int col = e < 4 ? c0 + e : c1 + (e - 4);
                  const bool in_slow = lgW == 3 ? true : ((gm >> (e >> 2)) & 1u) != 0;
                  const float val = (e & 1) ? A[4 * g + (e >> 1)].y : A[4 * g + (e >> 1)].x;
                  if (in_slow && col >= 0 && col < r.ncols) {
                    if (sub == 2) *reinterpret_cast<unsigned char*>(p + (long long)col) = (unsigned char)store_u8(val);
                    else *reinterpret_cast<uint32_t*>(p + (long long)col * 4) = store_i32(val);
                  }
                }
              }
            }
          }
        } break;
        case DVM_LK_STA: {
          const uint32_t a0 = sb + lean_opaque<16>(rec.y) + (uint32_t)tid * 16;
#pragma unroll
          for (int q = 0; q < V / 4; ++q)
            asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(a0 + q * PSTRIDE), "f"(A[2 * q].x), "f"(A[2 * q].y),
                         "f"(A[2 * q + 1].x), "f"(A[2 * q + 1].y)
                         : "memory");
        } break;
        case DVM_LK_LSS: {
          float v;
          asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(sb + lean_opaque<17>(rec.y) + (uint32_t)tid * 16));
          s_S[lean_opaque<57>(ra)][tid] = r.ncols > 0 ? v : 0.f;
        } break;
        case DVM_LK_STS: {
          bool first_block = r.col0 == 0;  // a row's value is stored once: by the tile of its first column block, or ...
          if constexpr (PHASED) {
            const uint32_t tag = rec.x >> 24;
            if (tag) {  // ... in a phased program by the last block of the phase that completes it
              if (tag - 1 != r.phase || !r.last_block) break;
              first_block = true;
            }
          }
          const uint32_t d = prog + lean_opaque<18>(rec.y);
          const int dt = (CW(d + DVM_OPD_INFO) >> 8) & 0xff;
          char* p = reinterpret_cast<char*>(tensor_ptr(prog, d) + (row_offset(prog, d, r) << DVM_DT_LG_ES(dt)));
          const float v = s_S[lean_opaque<58>(ra)][tid];
          if (r.ncols > 0 && t == 0 && first_block) {
            if (dt == DVM_DT_BF16) *reinterpret_cast<__nv_bfloat16*>(p) = __float2bfloat16_rn(v);
            else if (dt == DVM_DT_F32) *reinterpret_cast<float*>(p) = v;
            else if (dt == DVM_DT_I32) *reinterpret_cast<uint32_t*>(p) = store_i32(v);
            else *reinterpret_cast<unsigned char*>(p) = (unsigned char)store_u8(v);
          }
        } break;
        case DVM_LK_BCS: {
          const float v = s_S[lean_opaque<19>(ra)][tid];
          DVM_EACH_PAIR A[i] = make_float2(v, v);
        } break;
        case DVM_LK_CMP:
        case DVM_LK_SEL: {
          // Table 1, Cmp and Select (HEAVY variants): operands are fp32 images or temporaries, read in two halves
          if constexpr (HEAVY) {
            // half H of the register an operand word names (kind 1: fp32 image, 2: thread-private temporary) into pairs Y
#define DVM_LOAD_HALF(H, OW, KIND, Y)                                                                           \
            if ((KIND) == 2u) {                                                                                   \
              const uint32_t a_ = sb + ((OW) & 0x3ffffu) + (uint32_t)tid * 16;                                    \
              _Pragma("unroll") for (int q = 0; q < V / 8; ++q) {                                                 \
                const uint4 v = lean_lds128(a_ + (uint32_t)((H) * (V / 8) + q) * PSTRIDE);                        \
                Y[2 * q] = make_float2(__uint_as_float(v.x), __uint_as_float(v.y));                               \
                Y[2 * q + 1] = make_float2(__uint_as_float(v.z), __uint_as_float(v.w));                           \
              }                                                                                                   \
            } else {                                                                                              \
              const uint32_t a_ = opw_addr(OW);                                                                   \
              uint32_t R[V / 2];                                                                                  \
              if (lgW == 3) lean_raw_f32<2, (H) * (V / 16), ((H) + 1) * (V / 16), AL>(R, a_, (uint32_t)(G << 5));     \
              else lean_raw_f32<1, (H) * (V / 8), ((H) + 1) * (V / 8), AL>(R, a_, (uint32_t)(G << 4));                \
              _Pragma("unroll") for (int i = 0; i < VP / 2; ++i)                                                  \
                Y[i] = make_float2(__uint_as_float(R[2 * i]), __uint_as_float(R[2 * i + 1]));                     \
            }
            if (h == DVM_LK_CMP) {
#define DVM_CMP_HALF(H)                                                                                          \
              {                                                                                                   \
                float2 Y[VP / 2];                                                                                 \
                if (ra == 3u) { _Pragma("unroll") for (int i = 0; i < VP / 2; ++i) Y[i] = A[(H) * (VP / 2) + i]; } \
                else { DVM_LOAD_HALF(H, rec.y, ra, Y) }                                                           \
                _Pragma("unroll") for (int i = 0; i < VP / 2; ++i) {                                              \
                  float2& a = A[(H) * (VP / 2) + i];                                                              \
                  bool bx, by;                                                                                    \
                  switch (sub) {                                                                                  \
                    case DVM_C_GT: bx = a.x > Y[i].x; by = a.y > Y[i].y; break;                                   \
                    case DVM_C_GE: bx = a.x >= Y[i].x; by = a.y >= Y[i].y; break;                                 \
                    case DVM_C_LT: bx = a.x < Y[i].x; by = a.y < Y[i].y; break;                                   \
                    case DVM_C_LE: bx = a.x <= Y[i].x; by = a.y <= Y[i].y; break;                                 \
                    case DVM_C_EQ: bx = a.x == Y[i].x; by = a.y == Y[i].y; break;                                 \
                    default: bx = a.x != Y[i].x; by = a.y != Y[i].y; break;                                       \
                  }                                                                                               \
                  a = make_float2(bx ? 1.f : 0.f, by ? 1.f : 0.f);                                                \
                }                                                                                                 \
              }
              DVM_CMP_HALF(0)
              DVM_CMP_HALF(1)
#undef DVM_CMP_HALF
            } else if (sub == 3u) {  // ACC = ACC != 0 ? imm1 : imm2
              const float i1 = __uint_as_float(rec.y), i2 = __uint_as_float(rec.z);
              DVM_EACH_PAIR A[i] = make_float2(A[i].x != 0.f ? i1 : i2, A[i].y != 0.f ? i1 : i2);
            } else {
              // sub 0: ACC = ACC != 0 ? L[p] : L[q];  1: ACC = L[p] != 0 ? L[q] : ACC;  2: ACC = L[p] != 0 ? ACC : L[q]
              const uint32_t kp = ra & 3u, kq = (ra >> 2) & 3u;
#define DVM_SEL_HALF(H)                                                                                          \
              {                                                                                                   \
                float2 P[VP / 2], Q[VP / 2];                                                                      \
                DVM_LOAD_HALF(H, rec.y, kp, P)                                                                    \
                DVM_LOAD_HALF(H, rec.z, kq, Q)                                                                    \
                _Pragma("unroll") for (int i = 0; i < VP / 2; ++i) {                                              \
                  float2& a = A[(H) * (VP / 2) + i];                                                              \
                  if (sub == 0u) a = make_float2(a.x != 0.f ? P[i].x : Q[i].x, a.y != 0.f ? P[i].y : Q[i].y);     \
                  else if (sub == 1u) a = make_float2(P[i].x != 0.f ? Q[i].x : a.x, P[i].y != 0.f ? Q[i].y : a.y); \
                  else a = make_float2(P[i].x != 0.f ? a.x : Q[i].x, P[i].y != 0.f ? a.y : Q[i].y);               \
                }                                                                                                 \
              }
              DVM_SEL_HALF(0)
              DVM_SEL_HALF(1)
#undef DVM_SEL_HALF
            }
#undef DVM_LOAD_HALF
          } else {
            err = ST_BAD_CODE;
          }
        } break;
        case DVM_LK_PHASE: {
          if constexpr (PHASED) {
            if (r.phase < ra) stop = true;  // the tiles of the earlier phases end here
          }
        } break;
        case DVM_LK_SOP: {
          if constexpr (PHASED) {
            const uint32_t tag = rec.x >> 24;
            if (tag && (tag - 1 != r.phase || !r.last_block)) break;  // once, when its operands are complete
          }
          const uint32_t ry = lean_opaque<20>(rec.y);
          const int s1 = (ry >> 8) & 0xff, s2 = (ry >> 16) & 0xff, sop = ry & 0xff;
          const float x = s_S[s1][tid];
          float rv;
          if (sub == DVM_SK_FMAU) {
            rv = __fadd_rn(__fmul_rn(x, __uint_as_float(rec.z)), __uint_as_float(rec.w));
            if (sop != 0xff) rv = scalar_unary(sop, rv);
          } else if (sub == DVM_SK_UN) rv = scalar_unary(sop, x);
          else rv = scalar_arith(sop, x, sub == DVM_SK_BIN ? s_S[s2][tid] : __uint_as_float(rec.z));
          s_S[lean_opaque<60>(ra)][tid] = rv;
        } break;
        default:
          err = ST_BAD_CODE;
          break;
      }
      if constexpr (PHASED) {
        if (stop) break;
      }
      }
      if (err == ST_BAD_CODE) break;
    }

    prog_idx = next_prog_idx;
    tile = next;
    if (!one_slot) buf ^= 1;
  }
  cp_async_wait<0>();

  if (err && tid == 0) atomicMax(prm.status, err);
  if (use_queue) {
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      const unsigned done = atomicAdd(&prm.queue[1], 1u);
      if (done == gridDim.x - 1) {  // the last CTA to finish returns the queue to its resting state
        prm.queue[0] = 0u;
        prm.queue[1] = 0u;
        prm.queue[2] = 0u;
        __threadfence();
      }
    }
  }
#undef DVM_ARITH
#undef DVM_EACH_PAIR
#undef DVM_P0
#undef DVM_P1
#undef CW
}

}  // namespace dvm
