// Device half of the operator compiler: the virtual machine (Sec. 4.3, Algorithm 2)
// as a persistent sm_100a kernel.
//
// One CTA of 256 threads is one "core" of Algorithm 2.  The bytecode program(s)
// arrive as the kernel-parameter block; every warp fetches instruction words
// from that block through the constant bank (warp-uniform loads) and loops over
// the CTA's tiles.  A code body is [load section][compute section]:
//   * every global tile load is a TMA bulk copy (cp.async.bulk, global ->
//     shared, completion on an mbarrier) that lands the tile's bytes in local
//     memory exactly as they lie in global memory: an "image" of the tile's
//     rows.  A dense operand's tile is one contiguous byte range: one copy,
//     issued by one thread; other operands are copied row by row (the first
//     thread of each row issues its row); a row vector shared by all rows is
//     copied once per slot.  Copies start and end on 16-byte boundaries (the
//     enclosing aligned range is fetched), so any row alignment works.
//     A CTA holds two tile slots: the copies of tile i+1 -- of the same or of
//     another stacked program -- are issued when tile i starts, so the next
//     tile's HBM traffic is in flight during the whole compute of the current
//     one and costs the compute threads no instructions;
//   * the compute section is accumulator code: ACC is one register-resident tile
//     (V = 16 or 32 fp32 per thread, as float2 pairs so that add / mul / fma
//     issue as packed f32x2 instructions); other operands are read from the
//     images (or from thread-private temporaries) with 128-bit shared loads,
//     bf16 widened on the fly, or are per-row scalars S0..S7.
//
// Tile geometry (chosen per instance by the host's shape tiling):
//   G = 2^lgG threads share one row; a CTA holds 256/G rows per tile.
//   Every thread owns V element slots of a tile register; slot s maps to
//   column  (t + G*(s / W)) * W + (s % W) - shift  of the tile's column block,
//   t = thread index inside the row group, W = vector width in elements,
//   shift = misalignment of the row segment start, so that a thread's W-slot
//   chunk is a 16-byte aligned vector of the primary operand -- in global
//   memory and therefore in its image.  An operand whose rows are aligned
//   differently is read as the two covering aligned vectors and realigned in
//   registers.  Slots outside the row segment hold whatever the enclosing
//   vectors contain; reductions and stores mask them.
//
// Every wait on an mbarrier is bounded; a wait that runs out sets the status
// word to ST_TIMEOUT and the CTA leaves its tile loop.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dvm_format.h"
#include "dvm_launch.h"
#include "dvm_math.cuh"

namespace dvm {

constexpr int THREADS = DVM_VM_THREADS;
#ifndef DVM_VM_MIN_CTAS
#define DVM_VM_MIN_CTAS 2
#endif

template <int PW>
struct VMParams {
  uint32_t n_programs;
  uint32_t total_tiles;
  uint32_t n_words;      // words used in `words`
  uint32_t use_queue;    // 1: tiles beyond the first are claimed from the work queue
  uint32_t slot_bytes;   // bytes of one tile slot in local memory (the largest program's)
  uint32_t levels;       // 1: the directory has a third table, and tiles wait for the tiles of earlier levels;
                         // 2: one tile slot per CTA (slot_bytes = 0): no tile is loaded ahead, nothing is waited for
  uint32_t tile_begin;   // one-program launches: the first tile of the launch (tiles [tile_begin, total_tiles) run; a
                         // caller that pipelines host copies with execution launches a program in ranges of tiles)
  uint32_t row_tiles;    // a phased program (DVM_OP_PHASE; one-program launches of the views variant): the P * CB tiles a CTA
                         // takes a row through, in order, before it moves on to its next row; otherwise 0
                         // (the field also keeps `words` on a 16-byte boundary: linked records are loaded as vectors)
  unsigned int* status;  // device status word
  unsigned int* queue;   // [0] next tile to claim, [1] CTAs finished, [2] tiles completed (all zero between launches)
  uint32_t words[PW];    // [program word offsets (n)][tile prefix sums (n+1)][tiles before the program's level (n, if levels)][programs ...]
};

struct TileCtx {
  uint32_t prog;     // word offset of the tile's program in the parameter block
  int lgG, lgW;
  int shift;         // elements between the thread-0 chunk start and the row segment start
  int cbase;         // (t << lgW) - shift: column of this thread's slot 0
  int ov;            // thread 0 of a row only: its first `ov` slots hold the row's last columns (wrap-around, see make_ctx)
  int ncols;         // valid columns of this thread's row inside the column block (0: nothing to do)
  int nvalid;        // slots s >= 8 are valid iff s < nvalid (the valid slots of a thread form a prefix,
  uint32_t hm;       //   except in the first chunk of a misaligned row: bit s of hm covers slots 0..7)
  uint32_t fullmask; // bit j: chunk j lies entirely inside the row segment
  uint32_t partmask; // bit j: chunk j is cut by the segment's head or tail
  uint32_t row;      // row of the dominant (collapsed) shape (not clamped: rows past the end have ncols = 0)
  uint32_t col0;
  uint32_t flags;
  uint32_t phase;    // phased programs: the tile's phase, and whether its column block is the row's last
  bool last_block;
};

__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// ---- mbarrier + bulk copy ----
__device__ __forceinline__ void vm_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void vm_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void vm_mbar_arrive_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool vm_mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait (2 s of %globaltimer, and a poll cap): false when it ran out.
static __device__ __noinline__ bool vm_mbar_wait_slow(uint32_t bar, uint32_t parity) {
  unsigned long long t0, t1;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
  for (uint32_t spin = 0; spin < (1u << 27); ++spin) {
    if (vm_mbar_try(bar, parity)) return true;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
    if (t1 - t0 > 2000000000ull) break;
  }
  return false;
}
__device__ __forceinline__ bool vm_mbar_wait(uint32_t bar, uint32_t parity) {
  if (vm_mbar_try(bar, parity)) return true;
  return vm_mbar_wait_slow(bar, parity);
}
// Bounded wait until the grid-wide counter of completed tiles has reached `need` (acquire: what those tiles
// stored is visible afterwards).  Same limits as the barrier wait; false when it ran out.
static __device__ __noinline__ bool vm_wait_tiles_done(const unsigned int* counter, uint32_t need) {
  unsigned long long t0, t1;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
  for (uint32_t spin = 0; spin < (1u << 27); ++spin) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= need) return true;
    if ((spin & 15u) != 15u) continue;  // each poll is an L2 round trip: look at the clock now and then
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
    if (t1 - t0 > 2000000000ull) break;
  }
  return false;
}
// global -> shared bulk copy of `bytes` (a multiple of 16; both addresses 16-byte aligned), completion on `bar`
__device__ __forceinline__ void vm_bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src),
               "r"(bytes), "r"(bar)
               : "memory");
}

// Table 1, ViewLoad with a strided column dim, one thread's part: slot sl of the thread holds column
// cbase + (sl >> lgW << (lgG + lgW)) + (sl & (W - 1)) of the row (+ wrap when negative: the wrap-around slots
// of a misaligned row's first thread); valid columns are fetched from row + col * cstep_bytes, widened to
// fp32, into the thread-private layout (vector q of the thread at dst + q * 256 * 16).  fp32 elements travel
// as 4-byte asynchronous copies, bf16 elements through a register.  Out of line: the extended variants call it.
static __device__ __noinline__ void vm_gather(const char* row, unsigned long long cstep_bytes, int lg_es, uint32_t dst,
                                              int cbase, int lgW, int lgG, int wrap, int ncols, int V) {
  auto column = [&](int sl) -> int {
    int col = cbase + ((sl >> lgW) << (lgG + lgW)) + (sl & ((1 << lgW) - 1));
    if (col < 0) col += wrap;
    return (col < 0 || col >= ncols) ? -1 : col;
  };
  auto slot_addr = [&](int sl) -> uint32_t {
    return dst + (uint32_t)(sl >> 2) * (uint32_t)(DVM_VM_THREADS * 16) + (uint32_t)(sl & 3) * 4;
  };
  if (lg_es == 1) {
    // bf16 goes through registers: eight loads in flight at a time, then their stores
#pragma unroll 1
    for (int s0 = 0; s0 < V; s0 += 8) {
      unsigned short raw[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int col = column(s0 + k);
        raw[k] = col >= 0 ? *reinterpret_cast<const unsigned short*>(row + (unsigned long long)col * cstep_bytes) : (unsigned short)0;
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const float v = __uint_as_float((uint32_t)raw[k] << 16);
        asm volatile("st.shared.f32 [%0], %1;" ::"r"(slot_addr(s0 + k)), "f"(v) : "memory");
      }
    }
  } else {
#pragma unroll 1
    for (int sl = 0; sl < V; ++sl) {
      const int col = column(sl);
      if (col < 0) continue;
      asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(slot_addr(sl)), "l"(row + (unsigned long long)col * cstep_bytes) : "memory");
    }
  }
}

// One value into an fp32 result that many tiles combine: comb 1 sum, 2 max, 3 min (the result was pre-filled
// with the operation's identity).  Max / min order floats through their bit patterns: non-negative values as
// signed integers, negative ones as unsigned integers in reverse.
static __device__ __forceinline__ void vm_atomic_combine(float* a, float v, uint32_t comb) {
  if (comb == 1) {
    atomicAdd(a, v);
  } else if (comb == 2) {
    v += 0.0f;  // -0 -> +0
    if (v >= 0.f) atomicMax(reinterpret_cast<int*>(a), __float_as_int(v));
    else atomicMin(reinterpret_cast<unsigned int*>(a), __float_as_uint(v));
  } else {
    v += 0.0f;
    if (v >= 0.f) atomicMin(reinterpret_cast<int*>(a), __float_as_int(v));
    else atomicMax(reinterpret_cast<unsigned int*>(a), __float_as_uint(v));
  }
}

// The rows a warp holds (32 / G row groups of G threads, G <= 32, all landing on one result row) combined by a
// reduce-scatter: at the step with lane distance sh a lane keeps the lower or upper half of its slots (by its
// bit sh) and receives its partner's values for that half.  Afterwards the lane owns n_own = V * G / 32 combined
// slots, R[0 .. n_own), which are the tile slots first_slot + i.
template <int V, int COMB>
static __device__ __forceinline__ void vm_combine_rows(float (&R)[V], int lane, int G, int& first_slot, int& n_own) {
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) {
    const int half = V * sh / 32;  // the steps run from lane distance 16 down to G: the slots left halve each time
    if (sh >= G && half >= 1) {
      const bool up = (lane & sh) != 0;
#pragma unroll
      for (int i = 0; i < half; ++i) {
        const float keep = up ? R[i + half] : R[i];
        const float send = up ? R[i] : R[i + half];
        const float got = __shfl_xor_sync(0xffffffffu, send, sh);
        R[i] = COMB == 1 ? keep + got : (COMB == 2 ? fmaxf(keep, got) : fminf(keep, got));
      }
      if (up) first_slot += half;
      n_own = half;
    }
  }
}

// Table 1, Pow: the library's powf (special cases as IEEE pow), kept out of line: the extended interpreter
// variant calls it once per element instead of carrying V copies of it.
static __device__ __noinline__ float vm_pow(float a, float b) { return powf(a, b); }

// SINGLE: one program per launch (dvm_launch).  Its word offset in the parameter block is a compile-time
// constant, so header fields become direct constant-bank operands, and the work queue is compiled out.
// EXT: 1: the variant that also decodes Cmp / Select / Pow / IsFinite (launched when a program uses them:
// DVM_F_EXT_ISA); 2: that, plus gathered inputs and tile stores into strided views (DVM_F_VIEWS).  The basic
// variant (0) stays as compact as it is without them, and variant 1 without the view code.
// LEVELS: the stacked variant with in-kernel waits between dependent levels (dvm_launch_stacked_levels).
// CTAS: resident CTAs per SM the kernel is compiled for (2; 3 for the one-slot launches of the level-wait variant,
// whose CTAs wait for their own tile: a third CTA is worth more there than the registers it costs).
template <int V, int PW, bool SINGLE, int EXT, bool LEVELS = false, int CTAS = DVM_VM_MIN_CTAS>
__global__ void __launch_bounds__(THREADS, CTAS) dvm_vm_kernel(const __grid_constant__ VMParams<PW> prm) {
  constexpr bool VIEWS = EXT >= 2;
  constexpr uint32_t kSingleProg = 3;  // directory of a one-program launch: [offset][0][n_tiles]
  constexpr int VP = V / 2;            // float2 pairs per tile register
  constexpr int NST = V / 16;          // 16-element steps of a local-register operand
  constexpr int GRP = V >= 32 ? 2 : 1; // steps whose shared loads are issued together, ahead of their arithmetic
  constexpr uint32_t PSTRIDE = THREADS * 16;  // bytes between consecutive vectors of a thread-private register
  extern __shared__ __align__(16) uint32_t s_dyn[];
  __shared__ float s_red[2][THREADS / 32];
  __shared__ uint32_t s_next[2];
  __shared__ float s_S[DVM_MAX_SREGS][THREADS];  // per-row scalar registers S0..S7 of every thread
  __shared__ __align__(8) unsigned long long s_bar[2];  // "tile landed" barrier of each tile slot
  __shared__ volatile uint32_t s_abort;

  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  // one spare unit in front of the slots: a realigned read may touch the 16 bytes below an image
  const uint32_t local_base = static_cast<uint32_t>(__cvta_generic_to_shared(s_dyn)) + DVM_LOCAL_UNIT;
  const uint32_t bar0 = static_cast<uint32_t>(__cvta_generic_to_shared(s_bar));
  const uint32_t n_prog = SINGLE ? 1u : prm.n_programs;
  const bool use_queue = SINGLE ? false : prm.use_queue != 0;
  // dependent stacking: a tile of directory entry i reads what the tiles [0, CW(2n + 1 + i)) of the launch
  // store, so its loads start only after that many tiles are complete (the tiles of the earlier levels)
  constexpr bool levels = LEVELS && !SINGLE;
  // one tile slot (DVM_F_ONE_SLOT): both slots are the same memory, so a tile's loads start only when the
  // previous tile is done -- the hold-back of a level change, without its wait
  const bool one_slot = levels && prm.levels == 2;
#define CW(i) (prm.words[(i)])  /* one word of the parameter block: a constant-bank load at a warp-uniform index */

  if (tid == 0) {
    s_abort = 0;
    vm_mbar_init(bar0, THREADS);
    vm_mbar_init(bar0 + 8, THREADS);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  auto slot_base = [&](int slot) -> uint32_t { return local_base + (slot ? prm.slot_bytes : 0u); };

  // word offsets of a program's tables
  auto opd_base = [&](uint32_t prog) -> uint32_t { return prog + DVM_HDR_WORDS + 2 * (CW(prog + DVM_H_COUNTS) & 0xff); };
  auto lreg_base = [&](uint32_t prog) -> uint32_t { return opd_base(prog) + ((CW(prog + DVM_H_COUNTS) >> 16) & 0xff) * DVM_OPD_WORDS; };
  auto body_base = [&](uint32_t prog) -> uint32_t { return lreg_base(prog) + ((CW(prog + DVM_H_GEOM) >> 16) & 0xff); };

  // device address of the tensor an operand descriptor (word offset d) names
  auto tensor_ptr = [&](uint32_t prog, uint32_t d) -> unsigned long long {
    const uint32_t tp = prog + DVM_HDR_WORDS + 2 * (CW(d + DVM_OPD_INFO) & 0xff);
    return (unsigned long long)CW(tp) | ((unsigned long long)CW(tp + 1) << 32);
  };
  // element offset of this thread's row (plus the column block start) inside operand d
  // (strides are below 2^32 elements -- the host rejects larger ones: 32 x 32 -> 64-bit products)
  auto row_offset = [&](uint32_t d, const TileCtx& c) -> unsigned long long {
    uint32_t i0 = c.row;
    unsigned long long off = 0;
    if (c.flags & DVM_F_OUTER_DIMS) {  // row -> coordinates over the collapsed outer dims
      const uint32_t n0 = CW(c.prog + DVM_H_OUTER0), n1 = CW(c.prog + DVM_H_OUTER1);
      const uint32_t q = i0 / n0;
      i0 -= q * n0;
      const uint32_t i2 = q / n1;
      off = (unsigned long long)(q - i2 * n1) * CW(d + DVM_OPD_STRIDE1) + (unsigned long long)i2 * CW(d + DVM_OPD_STRIDE2);
    }
    off += (unsigned long long)i0 * CW(d + DVM_OPD_STRIDE0);
    if ((CW(d + DVM_OPD_INFO) >> 16) & 0xff) off += c.col0;
    return off;
  };

  // Tile id -> this thread's row of the tile (closed forms, no loops): all the load section needs.
  auto ctx_rows = [&](TileCtx& c, uint32_t prog, uint32_t local_tile) {
    c.prog = prog;
    const uint32_t geom = CW(prog + DVM_H_GEOM);
    c.lgG = geom & 0xff;
    const int W = (geom >> 8) & 0xff;
    c.lgW = W == 8 ? 3 : 2;
    c.flags = geom >> 24;
    const uint32_t CB = CW(prog + DVM_H_COL_BLOCKS);
    uint32_t rb = local_tile, cb = 0;
    if (CB > 1) { rb = local_tile / CB; cb = local_tile - rb * CB; }
    if constexpr (VIEWS && SINGLE) {
      c.phase = 0;
      c.last_block = true;
      if (prm.row_tiles) {  // tile -> (row, phase, column block): the row's tiles are consecutive, phase by phase
        rb = local_tile / prm.row_tiles;
        const uint32_t sub = local_tile - rb * prm.row_tiles;
        c.phase = sub / CB;
        cb = sub - c.phase * CB;
        c.last_block = cb == CB - 1;
      }
    }
    const uint32_t rows = CW(prog + DVM_H_ROWS_LO);  // the host rejects more than 2^32 - 1 rows per program
    const uint32_t row = rb * (uint32_t)(THREADS >> c.lgG) + (uint32_t)(tid >> c.lgG);
    const uint32_t ctile = CW(prog + DVM_H_COL_TILE);
    c.col0 = cb * ctile;
    const uint32_t cend = (row == rows - 1) ? CW(prog + DVM_H_LAST_ROW_COLS) : CW(prog + DVM_H_COLS);
    int nc = 0;
    if (row < rows && cend > c.col0) nc = (int)min(cend - c.col0, ctile);
    c.ncols = nc;
    c.row = row;
  };
  // The rest of the geometry: the row's shift and this thread's slot masks.  `c` still holds the previous
  // tile's masks on entry (prev_*: its program, segment length and shift): they are kept when nothing changed.
  // misalignment (in elements) of the row segment start of the primary operand: the tile's chunks follow it
  auto row_shift = [&](const TileCtx& c) -> int {
    if (c.flags & DVM_F_ALIGNED) return 0;
    const uint32_t prog = c.prog;
    const uint32_t d = opd_base(prog) + CW(prog + DVM_H_PRIMARY) * DVM_OPD_WORDS;
    const uint32_t lg_es = ((CW(d + DVM_OPD_INFO) >> 8) & 0xff) == DVM_DT_BF16 ? 1 : 2;
    const uint32_t base_el = (uint32_t)tensor_ptr(prog, d) >> lg_es;
    uint32_t off;
    if (c.flags & DVM_F_PRIMARY_DENSE) off = c.row * CW(prog + DVM_H_COLS) + c.col0;  // low bits are all that matter
    else off = (uint32_t)row_offset(d, c);
    return (int)((base_el + off) & (uint32_t)((1 << c.lgW) - 1));
  };
  auto ctx_masks = [&](TileCtx& c, uint32_t prev_prog, int prev_ncols, int prev_shift) {
    const uint32_t prog = c.prog;
    const int W = 1 << c.lgW;
    const int G = 1 << c.lgG;
    const int t = tid & (G - 1);
    const int nc = c.ncols;
    const int shift = row_shift(c);
    c.cbase = (t << c.lgW) - shift;
    c.shift = shift;
    if (prev_prog == prog && nc == prev_ncols && shift == prev_shift) return;  // same masks as the previous tile
    // In mapping coordinates the segment is [shift, shift + ncols); this thread owns chunks t, t+G, ...
    // The first nf of them are whole, the next one may be cut by the segment's end: a prefix of P slots.
    const int nch = V >> c.lgW;
    const int n2 = nc > 0 ? nc + shift : 0;
    const int avail = (n2 >> c.lgW) - t;                         // whole chunks of the row at or after chunk t
    int nf = avail > 0 ? ((avail + G - 1) >> c.lgG) : 0;         // those that belong to this thread
    nf = nf < nch ? nf : nch;
    int rem = nf < nch ? n2 - ((t + (nf << c.lgG)) << c.lgW) : 0;
    rem = rem > 0 ? (rem < W ? rem : W) : 0;
    const int P = (nf << c.lgW) + rem;
    uint32_t full = (nf >= 32) ? 0xffffffffu : ((1u << nf) - 1u);
    uint32_t part = rem > 0 ? (1u << nf) : 0u;
    uint32_t hm = P >= 8 ? 0xffu : ((1u << P) - 1u);
    int ov = 0;
    if (shift > 0 && t == 0 && nc > 0) {
      // head chunk of a misaligned row: slots [0, shift) lie before the segment.  A program encoded for
      // aligned rows that is run on a misaligned tensor may fill its whole capacity: the row's last
      // `ov` columns then have no slot of their own and wrap around into these head slots.
      ov = nc + shift - (V << c.lgG);
      ov = ov > 0 ? ov : 0;
      hm &= ~((1u << shift) - 1u);
      hm |= (1u << ov) - 1u;
      full &= ~1u;
      part |= 1u;
    }
    c.ov = ov;
    c.hm = hm;
    c.nvalid = P;
    c.fullmask = full;
    c.partmask = part;
  };
  auto slot_valid = [&](const TileCtx& c, int s) -> bool { return s < 8 ? ((c.hm >> s) & 1u) != 0 : s < c.nvalid; };

  // ---- load section of a tile: bulk copies into the images of slot `slot`, one arrival per thread ----
  auto issue_loads = [&](const TileCtx& c, int slot, bool first_of_program) {
    const uint32_t prog = SINGLE ? kSingleProg : c.prog;
    const uint32_t opd0 = opd_base(prog), lreg0 = lreg_base(prog), body0 = body_base(prog);
    const uint32_t load_words = CW(prog + DVM_H_LOAD_WORDS);
    const uint32_t bar = bar0 + 8 * slot;
    if (!(c.flags & DVM_F_LOADS_BY_ROW) && warp != 0) {  // thread 0 issues every copy of this program's tiles
      vm_mbar_arrive(bar);
      return;
    }
    const uint32_t sb = slot_base(slot);
    const int t = tid & ((1 << c.lgG) - 1);
    // When every copy of the tile is thread 0's (dense tiles, row vectors), the lanes of warp 0 take one load
    // instruction each, as thread 0 would: the warp walks the load section once, in parallel.  What the issuing warp
    // spends here, the other warps wait for at the tile's next barrier.
    const bool by_lane = !(c.flags & DVM_F_LOADS_BY_ROW);
    const uint32_t row0 = c.row - (uint32_t)(tid >> c.lgG);  // the tile's first row
    for (uint32_t pc = by_lane ? (uint32_t)lane : 0u; pc < (by_lane ? min((uint32_t)lane + 1u, load_words) : load_words); ++pc) {
      const uint32_t w0 = CW(body0 + pc);
      const uint32_t d = opd0 + DVM_INSN_B(w0) * DVM_OPD_WORDS;
      if (DVM_INSN_OP(w0) == DVM_OP_LDG) {
        const uint32_t lw = CW(lreg0 + (DVM_INSN_A(w0) & 0x7f));
        const uint32_t mode = (lw >> 16) & 0xf;
        uint32_t dst = sb + (lw & 0xffffu) * DVM_LOCAL_UNIT;
        const uint32_t lg_es = ((CW(d + DVM_OPD_INFO) >> 8) & 0xff) == DVM_DT_BF16 ? 1 : 2;
        unsigned long long a = 0, n_el = 0;
        bool mine = false;
        if (VIEWS && mode == DVM_LM_GATHER) {
          // Table 1, ViewLoad with a strided column dim: this thread fetches the elements of its own slots
          // (column of slot s as in the compute section), widened to fp32, into the private layout
          // (vector q of the thread at (q * 256 + tid) * 16).  fp32 elements travel as 4-byte async copies.
          const int shift = row_shift(c);
          const unsigned long long cs = CW(d + DVM_OPD_COLSTRIDE);
          const unsigned long long r0 = row_offset(d, c) - c.col0 + (unsigned long long)c.col0 * cs;
          // wrap-around slots of a misaligned row's first thread (see ctx_masks)
          const int ov = (shift > 0 && t == 0) ? c.ncols + shift - (V << c.lgG) : 0;
          vm_gather(reinterpret_cast<const char*>(tensor_ptr(prog, d)) + (r0 << lg_es), cs << lg_es, (int)lg_es,
                    dst + (uint32_t)tid * 16, (t << c.lgW) - shift, c.lgW, c.lgG, ov > 0 ? (V << c.lgG) : 0, c.ncols, V);
        } else if (VIEWS && mode == DVM_LM_TRANSPOSED) {
          // a transposed operand: thread j copies column j of the tile's column block -- the tile's rows of that
          // column are adjacent in memory (row stride 1), one strip of up to 256 / G elements
          const uint32_t rows = CW(prog + DVM_H_ROWS_LO);
          const uint32_t R = (uint32_t)(THREADS >> c.lgG);
          const uint32_t row0 = c.row - (uint32_t)(tid >> c.lgG);  // the tile's first row
          const uint32_t ncol_t = min(CW(prog + DVM_H_COLS) - c.col0, CW(prog + DVM_H_COL_TILE));
          if ((uint32_t)tid < ncol_t && row0 < rows) {
            mine = true;
            TileCtx c0 = c;
            c0.row = row0;
            a = row_offset(d, c0) - c.col0 + (unsigned long long)(c.col0 + (uint32_t)tid) * CW(d + DVM_OPD_COLSTRIDE);
            n_el = min(R, rows - row0);
            dst += (uint32_t)tid * DVM_STRIP_PITCH(R, 1u << lg_es);
          }
        } else if (mode == DVM_LM_BLOCK) {
          if (by_lane || tid == 0) {  // the tile's first row: the whole tile is one byte range from there
            mine = true;
            const uint32_t rows = CW(prog + DVM_H_ROWS_LO), C = CW(prog + DVM_H_COLS);
            const uint32_t R = (uint32_t)(THREADS >> c.lgG);
            const uint32_t rv = min(R, rows - row0);
            const uint32_t last = (row0 + rv == rows) ? CW(prog + DVM_H_LAST_ROW_COLS) : C;
            a = (unsigned long long)row0 * C;
            n_el = (unsigned long long)(rv - 1) * C + last;
          }
        } else if (mode == DVM_LM_ROWS) {
          if (t == 0 && c.ncols > 0) {
            mine = true;
            a = row_offset(d, c);
            n_el = (unsigned long long)c.ncols;
            dst += (uint32_t)(tid >> c.lgG) * DVM_ROW_PITCH(1 << c.lgG, V, 1u << lg_es);
          }
        } else {  // DVM_LM_BCAST: the same row for every tile of the program; DVM_LM_BCAST_TILE: of its column block
          if ((first_of_program || mode == DVM_LM_BCAST_TILE) && (by_lane || tid == 0)) {
            mine = true;
            a = c.col0;
            n_el = min(CW(prog + DVM_H_COLS) - c.col0, CW(prog + DVM_H_COL_TILE));
          }
        }
        if (mine) {
          const unsigned long long g0 = tensor_ptr(prog, d) + (a << lg_es);
          const unsigned long long gs = g0 & ~15ull, ge = (g0 + (n_el << lg_es) + 15ull) & ~15ull;
          const uint32_t bytes = (uint32_t)(ge - gs);
          asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
          vm_bulk_load(dst, reinterpret_cast<const void*>(gs), bytes, bar);
        }
      } else {  // DVM_OP_LDS: one value per row into scalar slot ia of this tile slot (thread-private)
        const int dt = (CW(d + DVM_OPD_INFO) >> 8) & 0xff;
        const char* p = reinterpret_cast<const char*>(tensor_ptr(prog, d) + (row_offset(d, c) << (dt == DVM_DT_BF16 ? 1 : 2)));
        const uint32_t w = (uint32_t)DVM_INSN_A(w0);
        const uint32_t dst = sb + (CW(prog + DVM_H_LOCAL2) & 0xffffu) * DVM_LOCAL_UNIT + (uint32_t)tid * 16 + (w >> 2) * PSTRIDE + (w & 3) * 4;
        if (c.ncols > 0) {
          if (dt == DVM_DT_BF16) {
            const float v = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(p));
            asm volatile("st.shared.f32 [%0], %1;" ::"r"(dst), "f"(v) : "memory");
          } else {
            cp_async4(dst, p);
          }
        }
      }
    }
    vm_mbar_arrive(bar);
  };

  float2 A[VP];
#pragma unroll
  for (int i = 0; i < VP; ++i) A[i] = make_float2(0.f, 0.f);

#define DVM_EACH_PAIR _Pragma("unroll") for (int i = 0; i < VP; ++i)

  // Where this thread's part of local register k (element type dt) lies in tile slot `buf`:
  // 16-byte vector u is at  (u & 1 ? a1 : a) + (u >> 1) * vA ;  mis != 0: the vectors are not 16-byte aligned.
  // tr_pitch != 0: a TRANSPOSED register -- the element of column col lies at a + col * tr_pitch (raw type: tr_bf16).
  struct RegView { uint32_t a, a1, vA, mis; bool image; uint32_t tr_pitch; bool tr_bf16; };
  auto reg_view = [&](const TileCtx& c, uint32_t prog, uint32_t opd0, uint32_t lreg0, int k, int dt, int buf) -> RegView {
    RegView r;
    const uint32_t lw = CW(lreg0 + k);
    const uint32_t mode = (lw >> 16) & 0xf;
    uint32_t a = slot_base(buf) + (lw & 0xffffu) * DVM_LOCAL_UNIT;
    r.tr_pitch = 0;
    r.tr_bf16 = false;
    if constexpr (VIEWS) {
      if (mode == DVM_LM_TRANSPOSED) {
        const uint32_t raw_dt = (CW(opd0 + (lw >> 24) * DVM_OPD_WORDS + DVM_OPD_INFO) >> 8) & 0xff;
        const uint32_t lg_raw = raw_dt == DVM_DT_BF16 ? 1u : 2u;
        // every strip starts on the same phase of a 16-byte word as the tensor itself (column stride, strip length
        // and outer strides are whole 16-byte units): the address modulo 16 patched in at launch
        r.a = a + ((lw >> 20) & 0xfu) + ((uint32_t)(tid >> c.lgG) << lg_raw);
        r.a1 = r.a;
        r.vA = 0;
        r.mis = 0;
        r.image = false;
        r.tr_pitch = DVM_STRIP_PITCH(THREADS >> c.lgG, 1u << lg_raw);
        r.tr_bf16 = raw_dt == DVM_DT_BF16;
        return r;
      }
    }
    if (mode == DVM_LM_PRIVATE || (VIEWS && mode == DVM_LM_GATHER)) {
      r.a = a + (uint32_t)tid * 16;
      r.a1 = r.a + PSTRIDE;
      r.vA = 2 * PSTRIDE;
      r.mis = 0;
      r.image = false;
      return r;
    }
    const uint32_t d = opd0 + (lw >> 24) * DVM_OPD_WORDS;
    const uint32_t lg_es = dt == DVM_DT_BF16 ? 1 : 2;
    const uint32_t base_lo = (lw >> 20) & 0xfu;  // the tensor address modulo 16 (patched in at launch)
    const uint32_t rr = (uint32_t)(tid >> c.lgG);
    uint32_t off;  // element offset (low bits suffice) of the image's first element inside the tensor
    if (mode == DVM_LM_BLOCK) {
      const uint32_t C = CW(prog + DVM_H_COLS);
      off = (c.row - rr) * C;  // the tile's first row
      a += (rr * C) << lg_es;
    } else if (mode == DVM_LM_ROWS) {
      off = (uint32_t)row_offset(d, c);
      a += rr * (((uint32_t)V << (c.lgG + lg_es)) + 32u);
    } else {
      off = c.col0;
    }
    a += ((base_lo + (off << lg_es)) & 15u) + ((uint32_t)c.cbase << lg_es);
    const uint32_t vstr = (1u << (c.lgG + c.lgW)) << lg_es;  // bytes from one chunk of the thread to its next
    const bool half = lg_es == 2 && c.lgW == 3;              // an fp32 chunk of 8 elements is two vectors
    r.a = a;
    r.a1 = a + (half ? 16u : vstr);
    r.vA = half ? vstr : 2 * vstr;
    r.mis = a & 15u;
    r.image = true;
    return r;
  };
  auto lds128 = [&](uint32_t addr) -> uint4 {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
  };
  // one 16-byte vector that starts `mis` bytes into an aligned word: the two covering words, realigned
  auto lds128_realign = [&](uint32_t addr, uint32_t mis) -> uint4 {
    const uint32_t b = addr - mis;
    const uint4 x = lds128(b), y = lds128(b + 16);
    const uint32_t woff = mis >> 2, sel = (mis & 2) ? 0x5432u : 0x3210u;
    uint32_t t0 = x.x, t1 = x.y, t2 = x.z, t3 = x.w, t4 = y.x, t5 = y.y;
    if (woff & 2) { t0 = x.z; t1 = x.w; t2 = y.x; t3 = y.y; t4 = y.z; t5 = y.w; }
    if (woff & 1) { t0 = t1; t1 = t2; t2 = t3; t3 = t4; t4 = t5; }
    return make_uint4(__byte_perm(t0, t1, sel), __byte_perm(t1, t2, sel), __byte_perm(t2, t3, sel), __byte_perm(t3, t4, sel));
  };
  auto widen_bf16 = [&](const uint4& v, float2* o) {
    o[0] = make_float2(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u));
    o[1] = make_float2(__uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
    o[2] = make_float2(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xffff0000u));
    o[3] = make_float2(__uint_as_float(v.w << 16), __uint_as_float(v.w & 0xffff0000u));
  };
  // D = L[k] widened to fp32: the whole tile register of this thread.  One warp-uniform branch picks the
  // variant (element type; aligned vectors or realigned ones); each variant is straight-line code.
  auto load_reg = [&](float2 (&D)[VP], const TileCtx& c, const RegView& r, int dt) {
    if constexpr (VIEWS) {
      if (r.tr_pitch) {
        // transposed strips: slot s holds column cbase + chunk offset (wrapped / clamped like a gathered slot:
        // slots outside the row read some strip of the image and are masked by their consumers)
        const int wrapcap = c.ov > 0 ? (V << c.lgG) : 0;
        const int last = max((int)CW((SINGLE ? kSingleProg : c.prog) + DVM_H_COL_TILE) - 1, 0);
#pragma unroll
        for (int sl = 0; sl < V; ++sl) {
          int col = c.cbase + ((sl >> c.lgW) << (c.lgG + c.lgW)) + (sl & ((1 << c.lgW) - 1));
          if (col < 0) col += wrapcap;
          col = min(max(col, 0), last);
          const uint32_t addr = r.a + (uint32_t)col * r.tr_pitch;
          float v;
          if (r.tr_bf16) {
            unsigned short h;
            asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(addr));
            v = __uint_as_float((uint32_t)h << 16);
          } else {
            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
          }
          if (sl & 1) D[sl >> 1].y = v; else D[sl >> 1].x = v;
        }
        return;
      }
    }
    const bool slow = __any_sync(0xffffffffu, r.mis != 0 || (c.ov > 0 && r.image));
    if (dt == DVM_DT_BF16) {
      if (!slow) {
#pragma unroll
        for (int u = 0; u < V / 8; ++u) widen_bf16(lds128(((u & 1) ? r.a1 : r.a) + (uint32_t)(u >> 1) * r.vA), &D[4 * u]);
      } else {
#pragma unroll
        for (int u = 0; u < V / 8; ++u)
          widen_bf16(lds128_realign(((u & 1) ? r.a1 : r.a) + (uint32_t)(u >> 1) * r.vA, r.mis), &D[4 * u]);
      }
    } else {
      if (!slow) {
#pragma unroll
        for (int u = 0; u < V / 4; ++u) {
          const uint4 v = lds128(((u & 1) ? r.a1 : r.a) + (uint32_t)(u >> 1) * r.vA);
          D[2 * u] = make_float2(__uint_as_float(v.x), __uint_as_float(v.y));
          D[2 * u + 1] = make_float2(__uint_as_float(v.z), __uint_as_float(v.w));
        }
      } else {
#pragma unroll
        for (int u = 0; u < V / 4; ++u) {
          const uint4 v = lds128_realign(((u & 1) ? r.a1 : r.a) + (uint32_t)(u >> 1) * r.vA, r.mis);
          D[2 * u] = make_float2(__uint_as_float(v.x), __uint_as_float(v.y));
          D[2 * u + 1] = make_float2(__uint_as_float(v.z), __uint_as_float(v.w));
        }
      }
    }
    if (slow && c.ov > 0 && r.image) {
      // wrap-around: the first `ov` slots are the columns one chunk past this thread's last chunk
      float2 e[4];
      const uint32_t wv = (uint32_t)(V >> (dt == DVM_DT_BF16 ? 3 : 2));  // vector index V * es / 16: one past the thread's last
      const uint32_t wa = ((wv & 1u) ? r.a1 : r.a) + (wv >> 1) * r.vA;
      const uint4 v0 = lds128_realign(wa, r.mis);
      if (dt == DVM_DT_BF16) {
        widen_bf16(v0, e);
      } else {
        // second half of an 8-element chunk; with chunks of 4 the address would be the NEXT chunk's, a sixth chunk that no
        // image holds -- past the end of the CTA's local memory when the register is the slot's last
        const uint4 v1 = lds128_realign(wa + (c.lgW == 3 ? r.a1 - r.a : 0u), r.mis);  // (chunks of 4: the first half again, unused)
        e[0] = make_float2(__uint_as_float(v0.x), __uint_as_float(v0.y));
        e[1] = make_float2(__uint_as_float(v0.z), __uint_as_float(v0.w));
        e[2] = make_float2(__uint_as_float(v1.x), __uint_as_float(v1.y));
        e[3] = make_float2(__uint_as_float(v1.z), __uint_as_float(v1.w));
      }
#pragma unroll
      for (int s2 = 0; s2 < 4; ++s2) {
        if (2 * s2 < c.ov) D[s2].x = e[s2].x;
        if (2 * s2 + 1 < c.ov) D[s2].y = e[s2].y;
      }
    }
  };

  uint32_t prog_idx = 0;
  uint32_t tile = blockIdx.x + (SINGLE ? prm.tile_begin : 0u);
  if constexpr (VIEWS && SINGLE) if (prm.row_tiles) tile = blockIdx.x * prm.row_tiles;
  uint32_t iter = 0;
  int red_par = 0;
  int buf = 0;
  unsigned err = 0;

  TileCtx c;
  c.prog = 0xffffffffu;
  c.ncols = -1;
  c.shift = 0;
  c.hm = c.fullmask = c.partmask = 0;
  c.nvalid = 0;
  c.ov = 0;
  uint32_t slot_prog[2] = {0xffffffffu, 0xffffffffu};  // program whose row-vector inputs each slot holds
  uint32_t published = 0;  // tiles of this CTA already counted in the grid-wide completion counter (of `iter` done)
  bool held = false;  // the current tile's loads are held back until the tiles of the earlier levels are complete
  if (tile < prm.total_tiles) {
    if (!SINGLE) while (prog_idx + 1 < n_prog && tile >= CW(n_prog + prog_idx + 1)) ++prog_idx;
    if (!SINGLE && levels && (one_slot || CW(2 * n_prog + 1 + prog_idx) > 0)) {
      held = true;
    } else {
      TileCtx cl;
      ctx_rows(cl, SINGLE ? kSingleProg : CW(prog_idx), SINGLE ? tile : tile - CW(n_prog + prog_idx));
      issue_loads(cl, buf, true);
      slot_prog[0] = prog_idx;
      cp_async_commit();
    }
  }

  while (tile < prm.total_tiles) {
    // ---- Algorithm 2, outer loop.  Every thread must be done with the previous tile before the other slot
    // is overwritten with the next tile's loads, which start now, ahead of the wait for this tile's bytes. ----
    if constexpr (levels) {
      if (held) {
        // This CTA moves on to a later level.  Behind the barrier the stores of its earlier tiles are all
        // issued: thread 0 publishes them (the fence is cumulative over what the barrier ordered before it)
        // and counts those tiles -- only here, and when the CTA ends: tiles of the level a CTA is still
        // working on are nobody's business yet, and a fence per tile would hold up thread 0, which issues the
        // next tile's copies.  Then it waits, before it claims anything further: a waiting CTA sits on one
        // tile only, the rest of the queue stays open to CTAs that are free.
        // All earlier tiles were claimed before this one, by CTAs that are resident (the grid never exceeds
        // the resident capacity) and that wait only for still earlier levels: the count gets there.
        __syncthreads();
        if (tid == 0 && !one_slot) {
          if (iter > published) {
            __threadfence();
            atomicAdd(&prm.queue[2], iter - published);
          }
          if (!vm_wait_tiles_done(&prm.queue[2], CW(2 * n_prog + 1 + prog_idx))) {
            err = ST_TIMEOUT;
            s_abort = 1;
          }
        }
        if (!one_slot) published = iter;
      }
    }
    if (use_queue && tid == 0) s_next[iter & 1] = atomicAdd(&prm.queue[0], 1u) + gridDim.x;
    __syncthreads();
    if (s_abort) break;  // a wait ran out in some thread during the previous tile
    if constexpr (levels) {
      {
        if (held) {
          asm volatile("fence.proxy.async;" ::: "memory");  // the bulk copies below read what generic stores wrote
          TileCtx cl;
          ctx_rows(cl, CW(prog_idx), tile - CW(n_prog + prog_idx));
          issue_loads(cl, buf, true);  // a held tile is this CTA's first of its program: earlier tiles were of earlier levels
          if (buf) slot_prog[1] = prog_idx; else slot_prog[0] = prog_idx;
          cp_async_commit();
          held = false;
        }
      }
    }
    uint32_t next = use_queue ? s_next[iter & 1] : tile + gridDim.x;
    if constexpr (VIEWS && SINGLE) {
      if (prm.row_tiles) {  // the next tile of this row, or the first tile of this CTA's next row
        next = tile + 1;
        if (next % prm.row_tiles == 0) next += (gridDim.x - 1) * prm.row_tiles;
      }
    }
    ++iter;
    const bool have_next = next < prm.total_tiles;
    uint32_t next_prog_idx = prog_idx;
    if (have_next) {
      if (!SINGLE) while (next_prog_idx + 1 < n_prog && next >= CW(n_prog + next_prog_idx + 1)) ++next_prog_idx;
      const uint32_t nprog = SINGLE ? kSingleProg : CW(next_prog_idx);
      const bool first = buf ? slot_prog[0] != next_prog_idx : slot_prog[1] != next_prog_idx;
      // the next tile belongs to a later level than this one: it also waits for this tile, so its loads
      // cannot start ahead (a tile of this tile's own level has nothing left to wait for)
      if (!SINGLE && levels && (one_slot || CW(2 * n_prog + 1 + next_prog_idx) > tile)) {
        held = true;
      } else if (((CW(nprog + DVM_H_GEOM) >> 24) & DVM_F_LOADS_BY_ROW) || warp == 0) {
        TileCtx cl;  // rows of the next tile, for the threads that may issue its copies
        ctx_rows(cl, nprog, SINGLE ? next : next - CW(n_prog + next_prog_idx));
        issue_loads(cl, buf ^ 1, first);
      } else {
        vm_mbar_arrive(bar0 + 8 * (buf ^ 1));  // thread 0 issues every copy of that program's tiles
      }
      if (buf) slot_prog[0] = next_prog_idx; else slot_prog[1] = next_prog_idx;
      cp_async_commit();
      cp_async_wait<1>();  // this tile's per-row scalars have landed once only the next tile's group is pending
    } else {
      cp_async_wait<0>();
    }
    if (!vm_mbar_wait(bar0 + 8 * buf, ((iter - 1) >> 1) & 1)) {
      // this tile's bytes did not land in time: report it, and leave the loop with everybody at the next
      // barrier; until then this thread keeps in step (the code it walks has the same barriers for all)
      err = ST_TIMEOUT;
      s_abort = 1;
    }
    {
      const uint32_t prev_prog = c.prog;
      const int prev_ncols = c.ncols, prev_shift = c.shift;
      ctx_rows(c, SINGLE ? kSingleProg : CW(prog_idx), SINGLE ? tile : tile - CW(n_prog + prog_idx));
      ctx_masks(c, prev_prog, prev_ncols, prev_shift);
    }

    const uint32_t prog = SINGLE ? kSingleProg : c.prog;
    const uint32_t opd0 = opd_base(prog), lreg0 = lreg_base(prog), body0 = body_base(prog);
    const uint32_t body_words = CW(prog + DVM_H_CODE_WORDS);
    const int W = 1 << c.lgW;
    const int G = 1 << c.lgG;
    const bool all_valid = __all_sync(0xffffffffu, c.nvalid == V && c.hm == 0xffu);

    // ---- Algorithm 2, inner loop: walk the compute section.  Two-level dispatch: the instruction class
    // (op >> 3) picks the handler through one jump table, the handler decodes only the fields it uses. ----
    uint32_t pc = body0 + CW(prog + DVM_H_LOAD_WORDS);
    const uint32_t pc_end = body0 + body_words;
    while (pc < pc_end) {
      const uint32_t w0 = CW(pc);
      const uint32_t op = DVM_INSN_OP(w0);
      switch (op >> 3) {
        case DVM_OP_BIN >> 3:
          if (DVM_INSN_A(w0) == DVM_REG_ACC) {  // ACC = ACC op ACC
            pc += 1;
            switch (op & 7) {
              case DVM_A_ADD: DVM_EACH_PAIR A[i] = __fadd2_rn(A[i], A[i]); break;
              case DVM_A_MUL: DVM_EACH_PAIR A[i] = __fmul2_rn(A[i], A[i]); break;
              case DVM_A_SUB: case DVM_A_RSUB: DVM_EACH_PAIR A[i] = __ffma2_rn(A[i], make_float2(-1.f, -1.f), A[i]); break;
              case DVM_A_DIV: case DVM_A_RDIV: DVM_EACH_PAIR A[i] = make_float2(fast_div(A[i].x, A[i].x), fast_div(A[i].y, A[i].y)); break;
              default: break;  // min / max of a value with itself
            }
            break;
          }
          // fall through: ACC = ACC op L[y]
        case DVM_OP_LD2 >> 3: {
          // ---- ACC = ACC op L[y]   (LD2: ACC = L[x] first) ----
          pc += 1;
          int ky = DVM_INSN_A(w0), dty = DVM_INSN_B(w0);
          if (op >= DVM_OP_LD2) {
            const int ib = DVM_INSN_B(w0);
            const int dtx = (ib >> 6) & 1;
            load_reg(A, c, reg_view(c, prog, opd0, lreg0, ky, dtx, buf), dtx);
            ky = ib & 0x3f;
            dty = (ib >> 7) & 1;
          }
          float2 Y[VP];
          load_reg(Y, c, reg_view(c, prog, opd0, lreg0, ky, dty, buf), dty);
          switch (op & 7) {
            case DVM_A_ADD: DVM_EACH_PAIR A[i] = __fadd2_rn(A[i], Y[i]); break;
            case DVM_A_SUB: DVM_EACH_PAIR A[i] = __ffma2_rn(Y[i], make_float2(-1.f, -1.f), A[i]); break;
            case DVM_A_RSUB: DVM_EACH_PAIR A[i] = __ffma2_rn(A[i], make_float2(-1.f, -1.f), Y[i]); break;
            case DVM_A_MUL: DVM_EACH_PAIR A[i] = __fmul2_rn(A[i], Y[i]); break;
            case DVM_A_DIV: DVM_EACH_PAIR A[i] = make_float2(fast_div(A[i].x, Y[i].x), fast_div(A[i].y, Y[i].y)); break;
            case DVM_A_RDIV: DVM_EACH_PAIR A[i] = make_float2(fast_div(Y[i].x, A[i].x), fast_div(Y[i].y, A[i].y)); break;
            case DVM_A_MIN: DVM_EACH_PAIR A[i] = make_float2(A[i].x < Y[i].x ? A[i].x : Y[i].x, A[i].y < Y[i].y ? A[i].y : Y[i].y); break;
            default: DVM_EACH_PAIR A[i] = make_float2(A[i].x > Y[i].x ? A[i].x : Y[i].x, A[i].y > Y[i].y ? A[i].y : Y[i].y); break;
          }
        } break;
        case DVM_OP_BINI >> 3:
        case DVM_OP_BINS >> 3: {
          // ---- ACC = ACC op y : y an immediate (word 1) or a per-row scalar ----
          float y;
          if (op >= DVM_OP_BINS) { y = s_S[DVM_INSN_A(w0)][tid]; pc += 1; }
          else { y = __uint_as_float(CW(pc + 1)); pc += 2; }
          const float2 y2 = make_float2(y, y);
          switch (op & 7) {
            case DVM_A_ADD: DVM_EACH_PAIR A[i] = __fadd2_rn(A[i], y2); break;
            case DVM_A_SUB: DVM_EACH_PAIR A[i] = __fadd2_rn(A[i], make_float2(-y, -y)); break;
            case DVM_A_RSUB: DVM_EACH_PAIR A[i] = __ffma2_rn(A[i], make_float2(-1.f, -1.f), y2); break;
            case DVM_A_MUL: DVM_EACH_PAIR A[i] = __fmul2_rn(A[i], y2); break;
            case DVM_A_DIV: {
              // division by a per-row scalar or an immediate: one SFU reciprocal (1 ulp), packed multiplies
              const float rcp = fast_rcp(y);
              DVM_EACH_PAIR A[i] = __fmul2_rn(A[i], make_float2(rcp, rcp));
            } break;
            case DVM_A_RDIV: DVM_EACH_PAIR A[i] = make_float2(fast_div(y, A[i].x), fast_div(y, A[i].y)); break;
            case DVM_A_MIN: DVM_EACH_PAIR A[i] = make_float2(A[i].x < y ? A[i].x : y, A[i].y < y ? A[i].y : y); break;
            default: DVM_EACH_PAIR A[i] = make_float2(A[i].x > y ? A[i].x : y, A[i].y > y ? A[i].y : y); break;
          }
        } break;
        case DVM_OP_UN >> 3:
        case (DVM_OP_UN >> 3) + 1: {
          pc += 1;
#define DVM_UN_CASE(U, EXPR)                                                          \
  case U:                                                                             \
    DVM_EACH_PAIR {                                                                   \
      float x = A[i].x; const float vx = (EXPR);                                      \
      x = A[i].y; const float vy = (EXPR);                                            \
      A[i] = make_float2(vx, vy);                                                     \
    }                                                                                 \
    break;
          switch (op - DVM_OP_UN) {
            DVM_UN_CASE(DVM_U_EXP, fast_exp(x))
            DVM_UN_CASE(DVM_U_SQRT, sqrtf(x))
            DVM_UN_CASE(DVM_U_RSQRT, rsqrtf(x))
            DVM_UN_CASE(DVM_U_ABS, fabsf(x))
            DVM_UN_CASE(DVM_U_LOG, logf(x))
            case DVM_U_ERF: DVM_EACH_PAIR A[i] = packed_erf(A[i]); break;
            DVM_UN_CASE(DVM_U_SIGMOID, fast_rcp(1.0f + fast_exp(-x)))
            DVM_UN_CASE(DVM_U_NEG, -x)
            DVM_UN_CASE(DVM_U_RECIP, fast_rcp(x))
            DVM_UN_CASE(DVM_U_FLOOR, floorf(x))
            DVM_UN_CASE(DVM_U_ROUND, rintf(x))
            DVM_UN_CASE(DVM_U_TANH, tanhf(x))
            DVM_UN_CASE(DVM_U_TRUNC_I32, trunc_i32(x))
            DVM_UN_CASE(DVM_U_TRUNC_U8, trunc_u8(x))
            default:
              if constexpr (EXT >= 1) {  // Table 1, IsFinite (programs that use it on a tile run the extended variant)
                if (op - DVM_OP_UN == DVM_U_ISFINITE) {
                  DVM_EACH_PAIR A[i] = make_float2(scalar_unary(DVM_U_ISFINITE, A[i].x), scalar_unary(DVM_U_ISFINITE, A[i].y));
                  break;
                }
              }
              DVM_EACH_PAIR A[i] = make_float2(round_bf16(A[i].x), round_bf16(A[i].y));
              break;
          }
#undef DVM_UN_CASE
        } break;
        case DVM_OP_ACT >> 3: {  // fused activations (pattern-based fusion, Sec. 5.1)
          pc += 1;
          if (op == DVM_OP_ACT + DVM_ACT_GELU) { DVM_EACH_PAIR A[i] = packed_gelu(A[i]); }
          else { DVM_EACH_PAIR A[i] = packed_silu(A[i]); }
        } break;
        case DVM_OP_RED >> 3: {
          // ---- row reduction (Table 1, Sum / Max / Min with N = 1): thread-local over valid slots, shuffles
          // inside the warp, shared memory across the warps of a row group ----
          pc += 1;
          const int rop = op & 7;
          bool accumulate = false;
          if constexpr (VIEWS && SINGLE) {
            const uint32_t tag = DVM_INSN_TAG(w0);
            if (tag) {  // a phased program: the reduction belongs to one phase and runs over that phase's blocks
              if (tag - 1 != c.phase) break;
              accumulate = c.col0 != 0;
            }
          }
          float v;
          if (rop == DVM_R_SUM || rop == DVM_R_SUMSQ) {
            // four partial sums per thread, pair i into sum i % 4 (as the lean interpreter: independent chains), then a tree
            float2 acc[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[q] = make_float2(0.f, 0.f);
            if (all_valid) {
              if (rop == DVM_R_SUM) { DVM_EACH_PAIR acc[i & 3] = __fadd2_rn(acc[i & 3], A[i]); }
              else { DVM_EACH_PAIR acc[i & 3] = __ffma2_rn(A[i], A[i], acc[i & 3]); }
            } else {
              DVM_EACH_PAIR {
                const float2 x = make_float2(slot_valid(c, 2 * i) ? A[i].x : 0.f, slot_valid(c, 2 * i + 1) ? A[i].y : 0.f);
                acc[i & 3] = rop == DVM_R_SUM ? __fadd2_rn(acc[i & 3], x) : __ffma2_rn(x, x, acc[i & 3]);
              }
            }
            const float2 a2 = __fadd2_rn(__fadd2_rn(acc[0], acc[1]), __fadd2_rn(acc[2], acc[3]));
            v = a2.x + a2.y;
#pragma unroll
            for (int sh = 1; sh < 32; sh <<= 1)
              if (sh < G) v += __shfl_xor_sync(0xffffffffu, v, sh);
          } else {
            const bool mx = rop == DVM_R_MAX;
            const float ident = mx ? -INFINITY : INFINITY;
            v = ident;
            if (all_valid) {
              DVM_EACH_PAIR v = mx ? fmaxf(v, fmaxf(A[i].x, A[i].y)) : fminf(v, fminf(A[i].x, A[i].y));
            } else {
              DVM_EACH_PAIR {
                const float x0 = slot_valid(c, 2 * i) ? A[i].x : ident;
                const float x1 = slot_valid(c, 2 * i + 1) ? A[i].y : ident;
                v = mx ? fmaxf(v, fmaxf(x0, x1)) : fminf(v, fminf(x0, x1));
              }
            }
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
            // only the warps of this row exchange partial results: a named barrier of their own (1 + row group)
            if (wpg == 8) __syncthreads();
            else asm volatile("bar.sync %0, %1;" ::"r"(1 + (warp >> (c.lgG - 5))), "r"(G) : "memory");
            const float* pr = &s_red[red_par][warp & ~(wpg - 1)];
            float x[8];
            x[0] = pr[0]; x[1] = pr[1];
            const float id2 = rop == DVM_R_MAX ? -INFINITY : (rop == DVM_R_MIN ? INFINITY : 0.f);
#pragma unroll
            for (int i = 2; i < 8; ++i) x[i] = id2;
            if (wpg > 2) { x[2] = pr[2]; x[3] = pr[3]; }
            if (wpg > 4) { x[4] = pr[4]; x[5] = pr[5]; x[6] = pr[6]; x[7] = pr[7]; }
            if (rop == DVM_R_MAX) v = fmaxf(fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3])), fmaxf(fmaxf(x[4], x[5]), fmaxf(x[6], x[7])));
            else if (rop == DVM_R_MIN) v = fminf(fminf(fminf(x[0], x[1]), fminf(x[2], x[3])), fminf(fminf(x[4], x[5]), fminf(x[6], x[7])));
            else v = ((x[0] + x[1]) + (x[2] + x[3])) + ((x[4] + x[5]) + (x[6] + x[7]));
            red_par ^= 1;
          }
          if constexpr (VIEWS && SINGLE) {
            if (accumulate) {
              const float prev = s_S[DVM_INSN_A(w0)][tid];
              v = rop == DVM_R_MAX ? fmaxf(prev, v) : (rop == DVM_R_MIN ? fminf(prev, v) : prev + v);
            }
          }
          s_S[DVM_INSN_A(w0)][tid] = v;
        } break;
        case 0: {  // NOP LDG LDS LDA STA LSS STG STS
          pc += 1;
          const int ia = DVM_INSN_A(w0), ib = DVM_INSN_B(w0);
          if (op == DVM_OP_LDA) {
            load_reg(A, c, reg_view(c, prog, opd0, lreg0, ia, ib, buf), ib);
          } else if (op == DVM_OP_STA) {
            const uint32_t a0 = slot_base(buf) + (CW(lreg0 + ia) & 0xffffu) * DVM_LOCAL_UNIT + (uint32_t)tid * 16;
#pragma unroll
            for (int q = 0; q < V / 4; ++q)
              asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(a0 + q * PSTRIDE), "f"(A[2 * q].x), "f"(A[2 * q].y),
                           "f"(A[2 * q + 1].x), "f"(A[2 * q + 1].y)
                           : "memory");
          } else if (op == DVM_OP_LSS) {
            const uint32_t w = (uint32_t)ib;
            float v;
            asm volatile("ld.shared.f32 %0, [%1];"
                         : "=f"(v)
                         : "r"(slot_base(buf) + (CW(prog + DVM_H_LOCAL2) & 0xffffu) * DVM_LOCAL_UNIT + (uint32_t)tid * 16 +
                               (w >> 2) * PSTRIDE + (w & 3) * 4));
            s_S[ia][tid] = c.ncols > 0 ? v : 0.f;
          } else if (op == DVM_OP_STG) {
            if constexpr (VIEWS && SINGLE) {
              if (DVM_INSN_TAG(w0) && DVM_INSN_TAG(w0) - 1 != c.phase) break;  // a phased program stores in its last phase
            }
            // an output covers the dominant shape: element (row, col) of a dense one lies at row * C + col,
            // the rows of a view (Table 1, ViewStore) lie where its strides put them
            const uint32_t d = opd0 + ib * DVM_OPD_WORDS;
            const uint32_t info = CW(d + DVM_OPD_INFO);
            const int dt = (info >> 8) & 0xff;
            const int lg_es = DVM_DT_LG_ES(dt);
            unsigned long long el0 = (unsigned long long)c.row * CW(prog + DVM_H_COLS) + c.col0;
            long long cstep = 1;  // elements between two columns of the output
            if constexpr (VIEWS) {  // programs with a strided output run the views variant (DVM_F_VIEWS)
              if (!((info >> 25) & 1u)) {
                cstep = (long long)CW(d + DVM_OPD_COLSTRIDE);
                el0 = row_offset(d, c) - c.col0 + (unsigned long long)c.col0 * (unsigned long long)cstep;
              }
            }
            char* p = reinterpret_cast<char*>(tensor_ptr(prog, d) + (el0 << lg_es));
            if constexpr (VIEWS) {
              const uint32_t comb = (info >> 26) & 3u;
              if (comb) {
                // A result that the tiles combine (a reduction over an axis the tiles walk along): the stored
                // view has stride 0 along that axis, so the rows of a tile land on one fp32 row of the result.
                // The rows a warp holds are combined by shuffles first when they share that row (32 / G row
                // groups per warp, G <= 32), then the warp's first row group issues the atomics.
                const bool row_ok = c.ncols > 0;
                bool uni = false;
                int colmax = c.ncols;
                unsigned long long el_out = el0;  // the result row this lane's atomics go to
                if (G <= 32) {
                  const unsigned long long first = __shfl_sync(0xffffffffu, el0, lane & (G - 1));
                  uni = __all_sync(0xffffffffu, !row_ok || el0 == first);
                  if (uni) {
                    // every lane writes combined slots, also lanes whose own row lies past the end: they all
                    // write to the row of the warp's first row group (rows ascend: it is valid if any is)
                    colmax = __shfl_sync(0xffffffffu, c.ncols, lane & (G - 1));
                    el_out = first;
                  }
                }
                const float ident = comb == 1 ? 0.f : (comb == 2 ? -INFINITY : INFINITY);
                float R[V];
#pragma unroll
                for (int sl = 0; sl < V; ++sl) {
                  const float a = (sl & 1) ? A[sl >> 1].y : A[sl >> 1].x;
                  R[sl] = slot_valid(c, sl) ? a : ident;  // (the slot masks of a row past the end are empty)
                }
                // reduce-scatter over the warp's row groups: at each step a lane keeps one half of its slots and
                // hands the other half to its partner, so every slot is combined once per step, not once per lane
                int first_slot = 0, n_own = V;
                if (uni) {
                  if (comb == 1) vm_combine_rows<V, 1>(R, lane, G, first_slot, n_own);
                  else if (comb == 2) vm_combine_rows<V, 2>(R, lane, G, first_slot, n_own);
                  else vm_combine_rows<V, 3>(R, lane, G, first_slot, n_own);
                }
                float* prow = reinterpret_cast<float*>(tensor_ptr(prog, d)) + el_out;
#pragma unroll
                for (int i = 0; i < V; ++i) {
                  if (i < n_own) {
                    const int sl = first_slot + i;
                    const int col = c.cbase + ((sl >> c.lgW) << (c.lgG + c.lgW)) + (sl & (W - 1));
                    if (col >= 0 && col < colmax && (uni || row_ok)) vm_atomic_combine(prow + (long long)col * cstep, R[i], comb);
                  }
                }
                break;
              }
            }
            char* q0 = p + ((long long)c.cbase << lg_es);
            const long long qstep = (long long)((G << c.lgW) << lg_es);
            // (a chunk of u8 is W bytes: its vector store wants that alignment; everything else goes in 16-byte vectors)
            const bool al = (reinterpret_cast<uintptr_t>(q0) & (dt == DVM_DT_U8 ? (uintptr_t)(W - 1) : (uintptr_t)15)) == 0 && (!VIEWS || cstep == 1);
            const uint32_t fast = al ? c.fullmask : 0u;
            const uint32_t slow = c.partmask | (c.fullmask & ~fast);
            constexpr uint32_t ALL8 = (V / 8 >= 32) ? 0xffffffffu : ((1u << (V / 8)) - 1u);
            if (dt == DVM_DT_BF16 && fast == ALL8) {  // every chunk whole and aligned: straight-line stores
  #pragma unroll
              for (int j = 0; j < V / 8; ++j) {
                uint32_t pk[4];
  #pragma unroll
                for (int q = 0; q < 4; ++q) {
                  const __nv_bfloat162 b = __floats2bfloat162_rn(A[4 * j + q].x, A[4 * j + q].y);
                  pk[q] = *reinterpret_cast<const uint32_t*>(&b);
                }
                *reinterpret_cast<uint4*>(q0 + j * qstep) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
              }
            } else if (dt == DVM_DT_BF16) {  // W == 8
  #pragma unroll
              for (int j = 0; j < V / 8; ++j) {
                if ((fast >> j) & 1) {
                  uint32_t pk[4];
  #pragma unroll
                  for (int q = 0; q < 4; ++q) {
                    const __nv_bfloat162 b = __floats2bfloat162_rn(A[4 * j + q].x, A[4 * j + q].y);
                    pk[q] = *reinterpret_cast<const uint32_t*>(&b);
                  }
                  *reinterpret_cast<uint4*>(q0 + j * qstep) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
              }
            } else if (dt == DVM_DT_U8) {  // Table 1, Cast: a chunk is W bytes
              if (W == 8) {
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
            } else if (dt == DVM_DT_I32) {
              if (W == 8) {
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
            } else if (W == 8) {
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
              // chunks cut by the segment's head or tail (or stored at another alignment than the mapping's):
              // pick the chunk's pairs out of ACC, then predicated element stores
  #pragma unroll 1
              for (uint32_t m = slow; m; m &= m - 1) {
                const int j = __ffs(m) - 1;
                float2 tp[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                if (W == 8) {
  #pragma unroll
                  for (int jj = 0; jj < V / 8; ++jj)
                    if (jj == j) { tp[0] = A[4 * jj]; tp[1] = A[4 * jj + 1]; tp[2] = A[4 * jj + 2]; tp[3] = A[4 * jj + 3]; }
                } else {
  #pragma unroll
                  for (int jj = 0; jj < V / 4; ++jj)
                    if (jj == j) { tp[0] = A[2 * jj]; tp[1] = A[2 * jj + 1]; }
                }
  #pragma unroll
                for (int el = 0; el < 8; ++el) {
                  if (el < W) {
                    int col = c.cbase + (j << (c.lgG + c.lgW)) + el;
                    if (col < 0 && c.ov > 0) col += V << c.lgG;  // wrap-around slots of the row's first thread
                    const float val = (el & 1) ? tp[el >> 1].y : tp[el >> 1].x;
                    if (col >= 0 && col < c.ncols) {
                      const long long ce = VIEWS ? (long long)col * cstep : (long long)col;  // scattered columns (Table 1, ViewStore)
                      if (dt == DVM_DT_BF16) *reinterpret_cast<__nv_bfloat16*>(p + ce * 2) = __float2bfloat16_rn(val);
                      else if (dt == DVM_DT_F32) *reinterpret_cast<float*>(p + ce * 4) = val;
                      else if (dt == DVM_DT_I32) *reinterpret_cast<uint32_t*>(p + ce * 4) = store_i32(val);
                      else *reinterpret_cast<unsigned char*>(p + ce) = (unsigned char)store_u8(val);
                    }
                  }
                }
              }
            }
          } else if (op == DVM_OP_STS) {
            bool first_block = c.col0 == 0;  // a row's value is stored once: by the tile of its first column block, or ...
            if constexpr (VIEWS && SINGLE) {
              const uint32_t tag = DVM_INSN_TAG(w0);
              if (tag) {  // ... in a phased program by the last block of the phase that completes it
                if (tag - 1 != c.phase || !c.last_block) break;
                first_block = true;
              }
            }
            const uint32_t d = opd0 + ib * DVM_OPD_WORDS;
            const int dt = (CW(d + DVM_OPD_INFO) >> 8) & 0xff;
            char* p = reinterpret_cast<char*>(tensor_ptr(prog, d) + (row_offset(d, c) << DVM_DT_LG_ES(dt)));
            const float v = s_S[ia][tid];
            if (c.ncols > 0 && (tid & (G - 1)) == 0 && first_block) {
              if (dt == DVM_DT_BF16) *reinterpret_cast<__nv_bfloat16*>(p) = __float2bfloat16_rn(v);
              else if (dt == DVM_DT_F32) *reinterpret_cast<float*>(p) = v;
              else if (dt == DVM_DT_I32) *reinterpret_cast<uint32_t*>(p) = store_i32(v);
              else *reinterpret_cast<unsigned char*>(p) = (unsigned char)store_u8(v);
            }
          } else if (op != DVM_OP_NOP) {
            err = ST_BAD_CODE;
            pc = pc_end;
          }
        } break;
        case 1: {  // BCS, SOP
          const int ia = DVM_INSN_A(w0), ib = DVM_INSN_B(w0);
          if (op == DVM_OP_BCS) {
            pc += 1;
            const float v = s_S[ia][tid];
            DVM_EACH_PAIR A[i] = make_float2(v, v);
          } else if (op == DVM_OP_PHASE) {
            pc += 1;
            if constexpr (VIEWS && SINGLE) {
              if (ia != 0xff && c.phase < (uint32_t)ia) pc = pc_end;  // the tiles of the earlier phases end here
            }
          } else if (op == DVM_OP_SOP) {
            if constexpr (VIEWS && SINGLE) {
              const uint32_t tag = DVM_INSN_TAG(w0);
              if (tag && (tag - 1 != c.phase || !c.last_block)) {  // phased: once, when its operands are complete
                pc += DVM_INSN_LEN(w0);
                break;
              }
            }
            const uint32_t w1 = CW(pc + 1);
            const int sub = w1 & 0xff, s1 = (w1 >> 8) & 0xff, s2 = (w1 >> 16) & 0xff;
            const float x = s_S[s1][tid];
            float rv;
            if (ib == DVM_SK_FMAU) {
              // unary(x * m + a): multiply and add round separately, exactly like the unfused instructions
              rv = __fadd_rn(__fmul_rn(x, __uint_as_float(CW(pc + 2))), __uint_as_float(CW(pc + 3)));
              if (sub != 0xff) rv = scalar_unary(sub, rv);
            } else if (ib == DVM_SK_UN) rv = scalar_unary(sub, x);
            else rv = scalar_arith(sub, x, ib == DVM_SK_BIN ? s_S[s2][tid] : __uint_as_float(CW(pc + 2)));
            s_S[ia][tid] = rv;
            pc += DVM_INSN_LEN(w0);
          } else {
            err = ST_BAD_CODE;
            pc = pc_end;
          }
        } break;
        case DVM_OP_CMP >> 3: if constexpr (EXT == 0) { err = ST_BAD_CODE; pc = pc_end; } else {
          // ---- ACC = ACC cmp L[y] ? 1 : 0   (Table 1, Cmp) ----
          pc += 1;
          const int ky = DVM_INSN_A(w0);
          float2 Y[VP];
          if (ky == DVM_REG_ACC) { DVM_EACH_PAIR Y[i] = A[i]; }
          else load_reg(Y, c, reg_view(c, prog, opd0, lreg0, ky, DVM_INSN_B(w0), buf), DVM_INSN_B(w0));
#define DVM_CMP_CASE(K, REL) \
  case K: DVM_EACH_PAIR A[i] = make_float2(A[i].x REL Y[i].x ? 1.f : 0.f, A[i].y REL Y[i].y ? 1.f : 0.f); break;
          switch (op & 7) {
            DVM_CMP_CASE(DVM_C_GT, >)
            DVM_CMP_CASE(DVM_C_GE, >=)
            DVM_CMP_CASE(DVM_C_LT, <)
            DVM_CMP_CASE(DVM_C_LE, <=)
            DVM_CMP_CASE(DVM_C_EQ, ==)
            // Table 1, Pow (unrolled calls of the out-of-line routine: ACC stays in registers)
            case DVM_C_POW: DVM_EACH_PAIR A[i] = make_float2(vm_pow(A[i].x, Y[i].x), vm_pow(A[i].y, Y[i].y)); break;
            case DVM_C_RPOW: DVM_EACH_PAIR A[i] = make_float2(vm_pow(Y[i].x, A[i].x), vm_pow(Y[i].y, A[i].y)); break;
            default: DVM_EACH_PAIR A[i] = make_float2(A[i].x != Y[i].x ? 1.f : 0.f, A[i].y != Y[i].y ? 1.f : 0.f); break;
          }
#undef DVM_CMP_CASE
        } break;
        case DVM_OP_SEL >> 3: if constexpr (EXT == 0) { err = ST_BAD_CODE; pc = pc_end; } else {
          // ---- Table 1, Select: the condition shrinks to one bit per slot; the value not in ACC streams in ----
          pc += 1;
          const int ib = DVM_INSN_B(w0);
          const int dt1 = (ib >> 6) & 1, dt2 = (ib >> 7) & 1;
          const int form = op & 7;
          if (form == 3) {  // ACC = ACC != 0 ? imm1 : imm2
            const float i1 = __uint_as_float(CW(pc)), i2 = __uint_as_float(CW(pc + 1));
            pc += 2;
            DVM_EACH_PAIR A[i] = make_float2(A[i].x != 0.f ? i1 : i2, A[i].y != 0.f ? i1 : i2);
            break;
          }
          float2 Y[VP];
          unsigned long long m = 0;
          if (form == 0) {  // ACC = ACC != 0 ? L[p] : L[q]
            DVM_EACH_PAIR m |= ((unsigned long long)(A[i].x != 0.f) << (2 * i)) | ((unsigned long long)(A[i].y != 0.f) << (2 * i + 1));
            load_reg(A, c, reg_view(c, prog, opd0, lreg0, DVM_INSN_A(w0), dt1, buf), dt1);
          } else {          // the condition is L[p]; 1: ACC = cond ? L[q] : ACC, 2: ACC = cond ? ACC : L[q]
            load_reg(Y, c, reg_view(c, prog, opd0, lreg0, DVM_INSN_A(w0), dt1, buf), dt1);
            DVM_EACH_PAIR m |= ((unsigned long long)(Y[i].x != 0.f) << (2 * i)) | ((unsigned long long)(Y[i].y != 0.f) << (2 * i + 1));
            if (form == 1) m = ~m;  // from here on: bit set = keep ACC
          }
          load_reg(Y, c, reg_view(c, prog, opd0, lreg0, ib & 0x3f, dt2, buf), dt2);
          DVM_EACH_PAIR A[i] = make_float2(((m >> (2 * i)) & 1) ? A[i].x : Y[i].x, ((m >> (2 * i + 1)) & 1) ? A[i].y : Y[i].y);
        } break;
        default:
          err = ST_BAD_CODE;
          pc = pc_end;  // stop walking code that cannot be decoded
          break;
      }
    }

    // ---- advance to the next tile ----
    prog_idx = next_prog_idx;
    tile = next;
    buf ^= 1;
  }
  cp_async_wait<0>();

  if (err && tid == 0) atomicMax(prm.status, err);
  if (use_queue) {
    // the last CTA to finish returns the queue to its resting state (all counters zero)
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      if (levels && iter > published) atomicAdd(&prm.queue[2], iter - published);  // this CTA's remaining tiles are complete
      const unsigned done = atomicAdd(&prm.queue[1], 1u);
      if (done == gridDim.x - 1) {
        prm.queue[0] = 0u;
        prm.queue[1] = 0u;
        prm.queue[2] = 0u;
        __threadfence();
      }
    }
  }
#undef DVM_EACH_PAIR
#undef CW
}

}  // namespace dvm
