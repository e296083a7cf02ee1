// Device half of the operator compiler: the virtual machine (Sec. 4.3, Algorithm 2)
// as a persistent sm_100a kernel.
//
// One CTA of 256 threads is one "core" of Algorithm 2.  The bytecode program(s)
// arrive as the kernel-parameter block; every warp fetches instruction words
// from that block through the constant bank (warp-uniform loads) and loops over
// the CTA's tiles.  A code body is [load section][compute section]:
//   * every global tile load is an asynchronous 16-byte global->shared copy
//     (cp.async) into a thread-private "local register" in shared memory -- the
//     paper's local memory.  A CTA holds two tile slots (complete register sets):
//     the load section of tile i+1 -- of the same or of another stacked program --
//     runs when tile i starts, so the next tile's HBM traffic is in flight during
//     the whole compute of the current one at no register cost; a row-vector
//     input of an aligned program is loaded once per slot;
//   * the compute section is accumulator code: ACC is one register-resident tile
//     (V = 16 or 32 fp32 per thread, as float2 pairs so that add / mul / fma
//     issue as packed f32x2 instructions); other operands are read from local
//     registers with 128-bit shared loads (bf16 operands widened on the fly), or
//     are per-row scalars S0..S7.
//
// Tile geometry (chosen per instance by the host's shape tiling):
//   G = 2^lgG threads share one row; a CTA holds 256/G rows per tile.
//   Every thread owns V element slots of a tile register; slot s maps to
//   column  (t + G*(s / W)) * W + (s % W) - shift  of the tile's column block,
//   t = thread index inside the row group, W = vector width in elements,
//   shift = misalignment of the row segment start, so that a thread's W-slot
//   chunk is a 16-byte aligned vector of the primary operand.  The `shift` slots
//   in front of the segment hold the segment's last columns (wrap-around), so a
//   row never needs more slots than it has columns.
// Whole chunks of an operand whose rows are aligned like the primary operand's
// are copied with cp.async; whole chunks at another alignment are fetched as the
// two covering aligned 16-byte words and realigned in registers; chunks cut by
// the segment's head or tail are assembled from predicated element loads.
//
// Local memory layout: units of 8 KB (32 bytes per thread); 16-byte vector q of a
// register at unit offset U lives at  U*8192 + (q * 256 + tid) * 16,
// i.e. consecutive threads touch consecutive vectors (no bank conflicts).
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
  uint32_t pad_;
  unsigned int* status;  // device status word
  unsigned int* queue;   // [0] next tile to claim, [1] CTAs finished (both zero between launches)
  uint32_t words[PW];    // [program word offsets][tile prefix sums (n+1)][programs ...]
};

struct TileCtx {
  uint32_t prog;     // word offset of the tile's program in the parameter block
  int t;             // thread index within the row group
  int lgG, lgW;
  int shift;
  int ncols;         // valid columns of this thread's row inside the column block (0: nothing to do)
  int nvalid;        // slots s >= 8 are valid iff s < nvalid (the valid slots of a thread form a prefix,
  uint32_t hm;       //   except in the first chunk of a misaligned row: bit s of hm covers slots 0..7)
  uint32_t fullmask; // bit j: chunk j lies entirely inside the row segment
  uint32_t partmask; // bit j: chunk j is cut by the segment's head or tail
  uint32_t i0, i1, i2;  // row coordinates over the collapsed outer dims
  uint32_t col0;
  uint32_t flags;
};

__device__ __forceinline__ float sget(const float (&S)[DVM_MAX_SREGS], int k) {
  float v = S[0];
#pragma unroll
  for (int i = 1; i < DVM_MAX_SREGS; ++i) v = (k == i) ? S[i] : v;
  return v;
}
__device__ __forceinline__ void sset(float (&S)[DVM_MAX_SREGS], int k, float v) {
#pragma unroll
  for (int i = 0; i < DVM_MAX_SREGS; ++i) S[i] = (k == i) ? v : S[i];
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// 16-byte copy when `on`, otherwise nothing is read (source size 0) and the destination is zero-filled
__device__ __forceinline__ void cp_async16_if(uint32_t dst, const void* src, bool on) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(on ? 16 : 0) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// SINGLE: one program per launch (dvm_launch).  Its word offset in the parameter block is a compile-time
// constant, so header fields become direct constant-bank operands, and the work queue is compiled out.
template <int V, int PW, bool SINGLE>
__global__ void __launch_bounds__(THREADS, DVM_VM_MIN_CTAS) dvm_vm_kernel(const __grid_constant__ VMParams<PW> prm) {
  constexpr uint32_t kSingleProg = 3;  // directory of a one-program launch: [offset][0][n_tiles]
  constexpr int VP = V / 2;            // float2 pairs per tile register
  constexpr int NST = V / 16;          // 16-element steps of a local-register operand
  constexpr int GRP = V >= 32 ? 2 : 1; // steps whose shared loads are issued together, ahead of their arithmetic
  constexpr uint32_t VSTRIDE = THREADS * 16;  // bytes between consecutive 16-byte vectors of a local register
  extern __shared__ __align__(16) uint32_t s_dyn[];
  __shared__ float s_red[2][THREADS / 32];
  __shared__ uint32_t s_next[2];

  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const uint32_t local_base = static_cast<uint32_t>(__cvta_generic_to_shared(s_dyn)) + (uint32_t)tid * 16;
  const uint32_t n_prog = SINGLE ? 1u : prm.n_programs;
  const bool use_queue = SINGLE ? false : prm.use_queue != 0;
#define CW(i) (prm.words[(i)])  /* one word of the parameter block: a constant-bank load at a warp-uniform index */

  // shared-memory address of 16-byte vector 0 of the register at unit offset U (this thread's part)
  auto lreg_addr = [&](uint32_t unit, int slot) -> uint32_t { return local_base + unit * DVM_LOCAL_UNIT + (slot ? prm.slot_bytes : 0u); };

  // word offsets of a program's tables
  auto opd_base = [&](uint32_t prog) -> uint32_t { return prog + DVM_HDR_WORDS + 2 * (CW(prog + DVM_H_COUNTS) & 0xff); };
  auto lreg_base = [&](uint32_t prog) -> uint32_t { return opd_base(prog) + ((CW(prog + DVM_H_COUNTS) >> 16) & 0xff) * DVM_OPD_WORDS; };
  auto body_base = [&](uint32_t prog) -> uint32_t { return lreg_base(prog) + ((CW(prog + DVM_H_GEOM) >> 16) & 0xff); };

  // Address of element (row, col0) of operand b -- or of the row's single value when col_stride = 0.
  auto operand_addr = [&](uint32_t prog, uint32_t opd0, int b, const TileCtx& c, int& dtype) -> char* {
    const uint32_t d = opd0 + b * DVM_OPD_WORDS;
    const uint32_t info = CW(d + DVM_OPD_INFO);
    const uint32_t tp = prog + DVM_HDR_WORDS + 2 * (info & 0xff);
    const unsigned long long base = (unsigned long long)CW(tp) | ((unsigned long long)CW(tp + 1) << 32);
    dtype = (info >> 8) & 0xff;
    // strides are below 2^32 elements (the host rejects larger ones): 32 x 32 -> 64-bit products
    unsigned long long off = (unsigned long long)c.i0 * CW(d + DVM_OPD_STRIDE0);
    if (c.flags & DVM_F_OUTER_DIMS) {
      off += (unsigned long long)c.i1 * CW(d + DVM_OPD_STRIDE1);
      off += (unsigned long long)c.i2 * CW(d + DVM_OPD_STRIDE2);
    }
    if ((info >> 16) & 0xff) off += c.col0;
    return reinterpret_cast<char*>(base + (off << (dtype == DVM_DT_BF16 ? 1 : 2)));
  };

  // Column (relative to the column block) of element e of chunk j, with the wrap-around of the head slots.
  auto chunk_col = [&](const TileCtx& c, int j, int e) -> int {
    const int col = ((c.t + (j << c.lgG)) << c.lgW) + e - c.shift;
    return col < 0 ? col + (V << c.lgG) : col;
  };

  // Tile id -> geometry of this thread's part of the tile (closed forms, no loops).
  auto make_ctx = [&](TileCtx& c, uint32_t prog, uint32_t local_tile) {
    c.prog = prog;
    const uint32_t geom = CW(prog + DVM_H_GEOM);
    c.lgG = geom & 0xff;
    const int W = (geom >> 8) & 0xff;
    c.lgW = W == 8 ? 3 : (W == 4 ? 2 : 0);
    c.flags = geom >> 24;
    const int G = 1 << c.lgG;
    c.t = tid & (G - 1);
    const uint32_t CB = CW(prog + DVM_H_COL_BLOCKS);
    uint32_t rb = local_tile, cb = 0;
    if (CB > 1) { rb = local_tile / CB; cb = local_tile - rb * CB; }
    const uint32_t rows = CW(prog + DVM_H_ROWS_LO);  // the host rejects more than 2^32 - 1 rows per program
    const uint32_t row = rb * (uint32_t)(THREADS >> c.lgG) + (uint32_t)(tid >> c.lgG);
    const uint32_t ctile = CW(prog + DVM_H_COL_TILE);
    c.col0 = cb * ctile;
    const uint32_t cend = (row == rows - 1) ? CW(prog + DVM_H_LAST_ROW_COLS) : CW(prog + DVM_H_COLS);
    int nc = 0;
    if (row < rows && cend > c.col0) nc = (int)min(cend - c.col0, ctile);
    c.ncols = nc;
    c.i0 = row < rows ? row : 0;
    c.i1 = c.i2 = 0;
    if (c.flags & DVM_F_OUTER_DIMS) {
      const uint32_t n0 = CW(prog + DVM_H_OUTER0), n1 = CW(prog + DVM_H_OUTER1);
      const uint32_t q = c.i0 / n0;
      c.i0 -= q * n0;
      c.i2 = q / n1;
      c.i1 = q - c.i2 * n1;
    }
    c.shift = 0;
    if (!(c.flags & DVM_F_ALIGNED) && W > 1) {
      const uint32_t pr = CW(prog + DVM_H_PRIMARY);
      if (pr != 0xffffffffu) {
        int dt;
        const unsigned long long a = reinterpret_cast<unsigned long long>(operand_addr(prog, opd_base(prog), (int)pr, c, dt));
        c.shift = (int)((a >> (dt == DVM_DT_BF16 ? 1 : 2)) & (unsigned long long)(W - 1));
      }
    }
    // In mapping coordinates the segment is [shift, shift + ncols); this thread owns chunks t, t+G, ...
    // The first nf of them are whole, the next one may be cut by the segment's end: a prefix of P slots.
    const int nch = V >> c.lgW;
    const int n2 = nc > 0 ? nc + c.shift : 0;
    const int avail = (n2 >> c.lgW) - c.t;                      // whole chunks of the row at or after chunk t
    int nf = avail > 0 ? ((avail + G - 1) >> c.lgG) : 0;         // those that belong to this thread
    nf = nf < nch ? nf : nch;
    int rem = nf < nch ? n2 - ((c.t + (nf << c.lgG)) << c.lgW) : 0;
    rem = rem > 0 ? (rem < W ? rem : W) : 0;
    const int P = (nf << c.lgW) + rem;
    uint32_t full = (nf >= 32) ? 0xffffffffu : ((1u << nf) - 1u);
    uint32_t part = rem > 0 ? (1u << nf) : 0u;
    uint32_t hm = P >= 8 ? 0xffu : ((1u << P) - 1u);
    if (c.shift > 0 && c.t == 0 && nc > 0) {
      // head chunk of a misaligned row: slots [0, shift) lie before the segment and hold its last
      // columns when the row fills the whole capacity (wrap-around)
      const int ov = nc + c.shift - (V << c.lgG);
      hm &= ~((1u << c.shift) - 1u);
      if (ov > 0) hm |= (1u << ov) - 1u;
      full &= ~1u;
      part |= 1u;
    }
    if (W == 1) { full = 0; part = 0; }  // element-wise mapping: the load / store paths count slots
    c.hm = hm;
    c.nvalid = P;
    c.fullmask = full;
    c.partmask = part;
  };
  auto slot_valid = [&](const TileCtx& c, int s) -> bool { return s < 8 ? ((c.hm >> s) & 1u) != 0 : s < c.nvalid; };

  // ---- one tile load (LDG instruction word w0) into buffer `buf` of its local register ----
  auto load_tile = [&](const TileCtx& c, uint32_t prog, uint32_t opd0, uint32_t lreg0, uint32_t w0, int buf) {
    const int ia = DVM_INSN_A(w0) & 0x7f, ib = DVM_INSN_B(w0);
    const int W = 1 << c.lgW;
    const int G = 1 << c.lgG;
    int dt;
    const char* p = operand_addr(prog, opd0, ib, c, dt);
    const uint32_t d0 = lreg_addr(CW(lreg0 + ia), buf);
    const int es = dt == DVM_DT_BF16 ? 2 : 4;
    if (W == 1) {
      // element-wise mapping: every valid slot is one scalar copy
#pragma unroll 1
      for (int sl = 0; sl < c.nvalid; ++sl) {
        const int col = c.t + (sl << c.lgG);
        const uint32_t b = (uint32_t)sl * es;
        const uint32_t dst = d0 + (b >> 4) * VSTRIDE + (b & 15);
        if (dt == DVM_DT_BF16) {
          const unsigned short hv = *reinterpret_cast<const unsigned short*>(p + (long long)col * 2);
          asm volatile("st.shared.u16 [%0], %1;" ::"r"(dst), "h"(hv) : "memory");
        } else {
          cp_async4(dst, p + (long long)col * 4);
        }
      }
      return;
    }
    const char* q0 = p + (long long)((c.t << c.lgW) - c.shift) * es;
    const long long qstep = (long long)(G << c.lgW) * es;
    const uint32_t mis = (uint32_t)(reinterpret_cast<uintptr_t>(q0) & 15);
    const uint32_t fast = mis ? 0u : c.fullmask;
    const uint32_t rea = mis ? c.fullmask : 0u;  // whole chunks at a misaligned address
    const int vpc = (W * es) >> 4;               // 16-byte vectors per chunk (1 or 2)
    if (fast && !c.partmask) {
      // every chunk of this thread is whole and aligned, or empty: one (bf16, fp32 W = 4) or two (fp32 W = 8)
      // 16-byte copies per chunk, switched off through the copy's source size (an empty chunk is zero-filled),
      // so that the chunk loop has no branches
      if (es == 2) {
#pragma unroll
        for (int j = 0; j < V / 8; ++j) cp_async16_if(d0 + j * VSTRIDE, q0 + j * qstep, (fast >> j) & 1);
      } else if (W == 8) {
#pragma unroll
        for (int j = 0; j < V / 8; ++j) {
          cp_async16_if(d0 + (2 * j) * VSTRIDE, q0 + j * qstep, (fast >> j) & 1);
          cp_async16_if(d0 + (2 * j + 1) * VSTRIDE, q0 + j * qstep + 16, (fast >> j) & 1);
        }
      } else {
#pragma unroll
        for (int j = 0; j < V / 4; ++j) cp_async16_if(d0 + j * VSTRIDE, q0 + j * qstep, (fast >> j) & 1);
      }
    } else if (fast) {
      // a chunk of this thread takes the element path below: copy only the whole ones (no zero fill may race with it)
#pragma unroll 1
      for (uint32_t m = fast; m; m &= m - 1) {
        const int j = __ffs(m) - 1;
        cp_async16(d0 + (j * vpc) * VSTRIDE, q0 + j * qstep);
        if (vpc == 2) cp_async16(d0 + (j * vpc + 1) * VSTRIDE, q0 + j * qstep + 16);
      }
    }
    if (rea) {
      // the operand's rows are aligned differently from the tile mapping: fetch the two aligned 16-byte
      // words that cover each vector and realign them in registers (word select + byte permute)
      const char* qa = q0 - mis;
      const uint32_t woff = mis >> 2, sel = (mis & 2) ? 0x5432u : 0x3210u;
#pragma unroll 1
      for (uint32_t m = rea; m; m &= m - 1) {
        const int j = __ffs(m) - 1;
        for (int v = 0; v < vpc; ++v) {
          const uint4 a = *reinterpret_cast<const uint4*>(qa + j * qstep + 16 * v);
          const uint4 bq = *reinterpret_cast<const uint4*>(qa + j * qstep + 16 * v + 16);
          uint32_t t0 = a.x, t1 = a.y, t2 = a.z, t3 = a.w, t4 = bq.x, t5 = bq.y;
          if (woff & 2) { t0 = a.z; t1 = a.w; t2 = bq.x; t3 = bq.y; t4 = bq.z; t5 = bq.w; }
          if (woff & 1) { t0 = t1; t1 = t2; t2 = t3; t3 = t4; t4 = t5; }
          const uint32_t o0 = __byte_perm(t0, t1, sel), o1 = __byte_perm(t1, t2, sel), o2 = __byte_perm(t2, t3, sel),
                         o3 = __byte_perm(t3, t4, sel);
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(d0 + (j * vpc + v) * VSTRIDE), "r"(o0), "r"(o1), "r"(o2), "r"(o3)
                       : "memory");
        }
      }
    }
    if (c.partmask) {
      // chunks cut by the row segment's head or tail: predicated element loads, one vector store
#pragma unroll 1
      for (uint32_t m = c.partmask; m; m &= m - 1) {
        const int j = __ffs(m) - 1;
        if (es == 2) {
          uint32_t h[8];
#pragma unroll
          for (int el = 0; el < 8; ++el) {
            const int col = chunk_col(c, j, el);
            h[el] = col < c.ncols ? (uint32_t)*reinterpret_cast<const unsigned short*>(p + (long long)col * 2) : 0u;
          }
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(d0 + j * VSTRIDE), "r"(h[0] | (h[1] << 16)),
                       "r"(h[2] | (h[3] << 16)), "r"(h[4] | (h[5] << 16)), "r"(h[6] | (h[7] << 16))
                       : "memory");
        } else {
          for (int v = 0; v < vpc; ++v) {
            uint32_t h[4];
#pragma unroll
            for (int el = 0; el < 4; ++el) {
              const int col = chunk_col(c, j, 4 * v + el);
              h[el] = col < c.ncols ? *reinterpret_cast<const uint32_t*>(p + (long long)col * 4) : 0u;
            }
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(d0 + (j * vpc + v) * VSTRIDE), "r"(h[0]), "r"(h[1]), "r"(h[2]),
                         "r"(h[3])
                         : "memory");
          }
        }
      }
    }
  };

  // ---- load section of a tile (the first tile of a program on this CTA also loads the tile-invariant inputs) ----
  auto issue_loads = [&](const TileCtx& c, int buf, bool first_of_program) {
    const uint32_t prog = SINGLE ? kSingleProg : c.prog;
    const uint32_t opd0 = opd_base(prog), lreg0 = lreg_base(prog), body0 = body_base(prog);
    const uint32_t load_words = CW(prog + DVM_H_LOAD_WORDS);
    for (uint32_t pc = 0; pc < load_words; ++pc) {
      const uint32_t w0 = CW(body0 + pc);
      if (DVM_INSN_OP(w0) == DVM_OP_LDG) {
        if ((DVM_INSN_A(w0) & 0x80) && !first_of_program) continue;  // tile-invariant operand: already in local memory
        load_tile(c, prog, opd0, lreg0, w0, buf);
      } else {  // DVM_OP_LDS: one value per row into scalar slot ia of this buffer
        int dt;
        const char* p = operand_addr(prog, opd0, DVM_INSN_B(w0), c, dt);
        const uint32_t unit = (CW(prog + DVM_H_LOCAL2) >> 8) & 0xff;
        const uint32_t w = (uint32_t)DVM_INSN_A(w0);
        const uint32_t dst = lreg_addr(unit, buf) + (w >> 2) * VSTRIDE + (w & 3) * 4;
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
  };

  float2 A[VP];
  float S[DVM_MAX_SREGS];
#pragma unroll
  for (int i = 0; i < DVM_MAX_SREGS; ++i) S[i] = 0.f;
#pragma unroll
  for (int i = 0; i < VP; ++i) A[i] = make_float2(0.f, 0.f);

#define DVM_EACH_PAIR _Pragma("unroll") for (int i = 0; i < VP; ++i)

  // reads 16 elements (step h) of the local register at address a0 (element type dt) into o[0..7] as fp32 pairs
  auto read_step = [&](float2 (&o)[8], uint32_t a0, int dt, int h) {
    if (dt == DVM_DT_BF16) {
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        uint4 v;
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a0 + (2 * h + q) * VSTRIDE));
        o[4 * q + 0] = make_float2(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u));
        o[4 * q + 1] = make_float2(__uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
        o[4 * q + 2] = make_float2(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xffff0000u));
        o[4 * q + 3] = make_float2(__uint_as_float(v.w << 16), __uint_as_float(v.w & 0xffff0000u));
      }
    } else {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float4 v;
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a0 + (4 * h + q) * VSTRIDE));
        o[2 * q] = make_float2(v.x, v.y);
        o[2 * q + 1] = make_float2(v.z, v.w);
      }
    }
  };
  // ACC = L[unit]
  auto read_acc = [&](uint32_t a0, int dt) {
#pragma unroll
    for (int h = 0; h < NST; ++h) {
      float2 o[8];
      read_step(o, a0, dt, h);
#pragma unroll
      for (int i = 0; i < 8; ++i) A[8 * h + i] = o[i];
    }
  };

  uint32_t prog_idx = 0;
  uint32_t tile = blockIdx.x;
  uint32_t iter = 0;
  int red_par = 0;
  int buf = 0;
  unsigned err = 0;

  TileCtx c;
  uint32_t slot_prog[2] = {0xffffffffu, 0xffffffffu};  // program whose tile-invariant inputs each slot holds
  if (tile < prm.total_tiles) {
    if (!SINGLE) while (prog_idx + 1 < n_prog && tile >= CW(n_prog + prog_idx + 1)) ++prog_idx;
    make_ctx(c, SINGLE ? kSingleProg : CW(prog_idx), SINGLE ? tile : tile - CW(n_prog + prog_idx));
    issue_loads(c, buf, true);
    slot_prog[0] = prog_idx;
    cp_async_commit();
  }

  while (tile < prm.total_tiles) {
    // ---- Algorithm 2, outer loop: next tile of this core; its loads start now, into the other tile slot ----
    uint32_t next;
    if (use_queue) {
      if (tid == 0) s_next[iter & 1] = atomicAdd(&prm.queue[0], 1u) + gridDim.x;
      __syncthreads();
      next = s_next[iter & 1];
    } else {
      next = tile + gridDim.x;
    }
    ++iter;
    TileCtx cn = c;
    const bool have_next = next < prm.total_tiles;
    uint32_t next_prog_idx = prog_idx;
    if (have_next) {
      if (!SINGLE) while (next_prog_idx + 1 < n_prog && next >= CW(n_prog + next_prog_idx + 1)) ++next_prog_idx;
      make_ctx(cn, SINGLE ? kSingleProg : CW(next_prog_idx), SINGLE ? next : next - CW(n_prog + next_prog_idx));
      const bool first = buf ? slot_prog[0] != next_prog_idx : slot_prog[1] != next_prog_idx;
      issue_loads(cn, buf ^ 1, first);
      if (buf) slot_prog[0] = next_prog_idx; else slot_prog[1] = next_prog_idx;
      cp_async_commit();
      cp_async_wait<1>();  // this tile's loads have landed once only the next tile's group is pending
    } else {
      cp_async_wait<0>();
    }

    const uint32_t prog = SINGLE ? kSingleProg : c.prog;
    const uint32_t opd0 = opd_base(prog), lreg0 = lreg_base(prog), body0 = body_base(prog);
    const uint32_t body_words = CW(prog + DVM_H_CODE_WORDS);
    const int W = 1 << c.lgW;
    const int G = 1 << c.lgG;
    const bool all_valid = __all_sync(0xffffffffu, c.nvalid == V && c.hm == 0xffu);

    // ---- Algorithm 2, inner loop: walk the compute section ----
    uint32_t pc = CW(prog + DVM_H_LOAD_WORDS);
    while (pc < body_words) {
      const uint32_t w0 = CW(body0 + pc);
      const uint32_t op = DVM_INSN_OP(w0);
      const int ia = DVM_INSN_A(w0), ib = DVM_INSN_B(w0);
      pc += max(DVM_INSN_LEN(w0), 1u);  // Insn_Len (Algorithm 2); the host verifier rejects 0

      if ((op >= DVM_OP_BIN && op < DVM_OP_BINS && ia != DVM_REG_ACC) || op >= DVM_OP_LD2) {
        // ---- ACC = ACC op L[y]   (LD2: ACC = L[x] first) -- the operand streams from local memory 16 elements
        // at a time ----
        uint32_t ay;
        int dty;
        if (op >= DVM_OP_LD2) {
          read_acc(lreg_addr(CW(lreg0 + ia), buf), (ib >> 6) & 1);
          ay = lreg_addr(CW(lreg0 + (ib & 0x3f)), buf);
          dty = (ib >> 7) & 1;
        } else {
          ay = lreg_addr(CW(lreg0 + ia), buf);
          dty = ib;
        }
#define DVM_TILE_OP(...)                                             \
  _Pragma("unroll") for (int g2 = 0; g2 < NST; g2 += GRP) {          \
    float2 o[GRP][8];                                                \
    _Pragma("unroll") for (int h = 0; h < GRP; ++h) read_step(o[h], ay, dty, g2 + h); \
    _Pragma("unroll") for (int h = 0; h < GRP; ++h)                  \
      _Pragma("unroll") for (int i = 0; i < 8; ++i) {                \
        float2& a = A[8 * (g2 + h) + i];                             \
        const float2 y = o[h][i];                                    \
        __VA_ARGS__                                                  \
      }                                                              \
  }
        switch (op & 7) {
          case DVM_A_ADD: DVM_TILE_OP(a = __fadd2_rn(a, y);) break;
          case DVM_A_SUB: DVM_TILE_OP(a = __ffma2_rn(y, make_float2(-1.f, -1.f), a);) break;
          case DVM_A_RSUB: DVM_TILE_OP(a = __ffma2_rn(a, make_float2(-1.f, -1.f), y);) break;
          case DVM_A_MUL: DVM_TILE_OP(a = __fmul2_rn(a, y);) break;
          case DVM_A_DIV: DVM_TILE_OP(a = make_float2(fast_div(a.x, y.x), fast_div(a.y, y.y));) break;
          case DVM_A_RDIV: DVM_TILE_OP(a = make_float2(fast_div(y.x, a.x), fast_div(y.y, a.y));) break;
          case DVM_A_MIN: DVM_TILE_OP(a = make_float2(a.x < y.x ? a.x : y.x, a.y < y.y ? a.y : y.y);) break;
          default: DVM_TILE_OP(a = make_float2(a.x > y.x ? a.x : y.x, a.y > y.y ? a.y : y.y);) break;
        }
#undef DVM_TILE_OP
        continue;
      }
      if (op >= DVM_OP_BINI && op < DVM_OP_UN) {
        // ---- ACC = ACC op y : y an immediate, a per-row scalar, or ACC itself ----
        if (op >= DVM_OP_BIN && op < DVM_OP_BINS) {  // ACC op ACC
          switch (op & 7) {
            case DVM_A_ADD: DVM_EACH_PAIR A[i] = __fadd2_rn(A[i], A[i]); break;
            case DVM_A_MUL: DVM_EACH_PAIR A[i] = __fmul2_rn(A[i], A[i]); break;
            case DVM_A_SUB: case DVM_A_RSUB: DVM_EACH_PAIR A[i] = __ffma2_rn(A[i], make_float2(-1.f, -1.f), A[i]); break;
            case DVM_A_DIV: case DVM_A_RDIV: DVM_EACH_PAIR A[i] = make_float2(fast_div(A[i].x, A[i].x), fast_div(A[i].y, A[i].y)); break;
            default: break;  // min / max of a value with itself
          }
          continue;
        }
        const float y = op >= DVM_OP_BINS ? sget(S, ia) : __uint_as_float(CW(body0 + pc - 1));
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
        continue;
      }
      if (op >= DVM_OP_UN && op < DVM_OP_RED) {
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
          DVM_UN_CASE(DVM_U_ERF, erff(x))
          DVM_UN_CASE(DVM_U_SIGMOID, fast_rcp(1.0f + fast_exp(-x)))
          DVM_UN_CASE(DVM_U_NEG, -x)
          DVM_UN_CASE(DVM_U_RECIP, fast_rcp(x))
          DVM_UN_CASE(DVM_U_FLOOR, floorf(x))
          DVM_UN_CASE(DVM_U_ROUND, rintf(x))
          DVM_UN_CASE(DVM_U_TANH, tanhf(x))
          default:
            DVM_EACH_PAIR A[i] = make_float2(round_bf16(A[i].x), round_bf16(A[i].y));
            break;
        }
#undef DVM_UN_CASE
        continue;
      }
      if (op >= DVM_OP_RED && op < DVM_OP_LD2) {
        // ---- row reduction (Table 1, Sum / Max / Min with N = 1): thread-local over valid slots, shuffles
        // inside the warp, shared memory across the warps of a row group ----
        const int rop = op - DVM_OP_RED;
        float v;
        if (rop == DVM_R_SUM || rop == DVM_R_SUMSQ) {
          float2 acc = make_float2(0.f, 0.f);
          if (all_valid) {
            if (rop == DVM_R_SUM) { DVM_EACH_PAIR acc = __fadd2_rn(acc, A[i]); }
            else { DVM_EACH_PAIR acc = __ffma2_rn(A[i], A[i], acc); }
          } else {
            DVM_EACH_PAIR {
              const float2 x = make_float2(slot_valid(c, 2 * i) ? A[i].x : 0.f, slot_valid(c, 2 * i + 1) ? A[i].y : 0.f);
              acc = rop == DVM_R_SUM ? __fadd2_rn(acc, x) : __ffma2_rn(x, x, acc);
            }
          }
          v = acc.x + acc.y;
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
#pragma unroll
          for (int sh = 1; sh < 32; sh <<= 1)
            if (sh < G) {
              const float x = __shfl_xor_sync(0xffffffffu, v, sh);
              v = mx ? fmaxf(v, x) : fminf(v, x);
            }
        }
        if (G > 32) {
          if (lane == 0) s_red[red_par][warp] = v;
          __syncthreads();
          const int wpg = G >> 5;  // warps per row group
          const int w0i = warp & ~(wpg - 1);
          float acc = s_red[red_par][w0i];
          for (int i = 1; i < wpg; ++i) {
            const float x = s_red[red_par][w0i + i];
            acc = rop == DVM_R_MAX ? fmaxf(acc, x) : (rop == DVM_R_MIN ? fminf(acc, x) : acc + x);
          }
          v = acc;
          red_par ^= 1;
        }
        sset(S, ia, v);
        continue;
      }

      switch (op) {
        case DVM_OP_NOP: break;
        case DVM_OP_LDA: {
          read_acc(lreg_addr(CW(lreg0 + ia), buf), ib);
        } break;
        case DVM_OP_STA: {
          const uint32_t a0 = lreg_addr(CW(lreg0 + ia), buf);
#pragma unroll
          for (int q = 0; q < V / 4; ++q)
            asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(a0 + q * VSTRIDE), "f"(A[2 * q].x), "f"(A[2 * q].y),
                         "f"(A[2 * q + 1].x), "f"(A[2 * q + 1].y)
                         : "memory");
        } break;
        case DVM_OP_LSS: {
          const uint32_t unit = (CW(prog + DVM_H_LOCAL2) >> 8) & 0xff;
          const uint32_t w = (uint32_t)ib;
          float v;
          asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(lreg_addr(unit, buf) + (w >> 2) * VSTRIDE + (w & 3) * 4));
          sset(S, ia, c.ncols > 0 ? v : 0.f);
        } break;
        case DVM_OP_STG: {
          int dt;
          char* p = operand_addr(prog, opd0, ib, c, dt);
          const int es = dt == DVM_DT_BF16 ? 2 : 4;
          if (W == 1) {
            // element-wise mapping: one predicated scalar store per slot
#pragma unroll
            for (int sl = 0; sl < V; ++sl) {
              if (sl < c.nvalid) {
                const long long col = c.t + (sl << c.lgG);
                const float val = (sl & 1) ? A[sl >> 1].y : A[sl >> 1].x;
                if (dt == DVM_DT_BF16) *reinterpret_cast<__nv_bfloat16*>(p + col * 2) = __float2bfloat16_rn(val);
                else *reinterpret_cast<float*>(p + col * 4) = val;
              }
            }
            break;
          }
          char* q0 = p + (long long)((c.t << c.lgW) - c.shift) * es;
          const long long qstep = (long long)(G << c.lgW) * es;
          const bool al = (reinterpret_cast<uintptr_t>(q0) & 15) == 0;
          const uint32_t fast = al ? c.fullmask : 0u;
          const uint32_t slow = c.partmask | (c.fullmask & ~fast);
          if (dt == DVM_DT_BF16) {  // W == 8
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
                  const int col = chunk_col(c, j, el);
                  const float val = (el & 1) ? tp[el >> 1].y : tp[el >> 1].x;
                  if (col < c.ncols) {
                    if (dt == DVM_DT_BF16) *reinterpret_cast<__nv_bfloat16*>(p + (long long)col * 2) = __float2bfloat16_rn(val);
                    else *reinterpret_cast<float*>(p + (long long)col * 4) = val;
                  }
                }
              }
            }
          }
        } break;
        case DVM_OP_STS: {
          int dt;
          char* p = operand_addr(prog, opd0, ib, c, dt);
          const float v = sget(S, ia);
          if (c.ncols > 0 && c.t == 0 && c.col0 == 0) {
            if (dt == DVM_DT_BF16) *reinterpret_cast<__nv_bfloat16*>(p) = __float2bfloat16_rn(v);
            else *reinterpret_cast<float*>(p) = v;
          }
        } break;
        case DVM_OP_BCS: {
          const float v = sget(S, ia);
          DVM_EACH_PAIR A[i] = make_float2(v, v);
        } break;
        case DVM_OP_SOP: {
          const uint32_t w1 = CW(body0 + pc - (ib == DVM_SK_BINI ? 2 : (ib == DVM_SK_FMAU ? 3 : 1)));
          const int sub = w1 & 0xff, s1 = (w1 >> 8) & 0xff, s2 = (w1 >> 16) & 0xff;
          const float x = sget(S, s1);
          float rv;
          if (ib == DVM_SK_FMAU) {
            // unary(x * m + a): multiply and add round separately, exactly like the unfused instructions
            rv = __fadd_rn(__fmul_rn(x, __uint_as_float(CW(body0 + pc - 2))), __uint_as_float(CW(body0 + pc - 1)));
            if (sub != 0xff) rv = scalar_unary(sub, rv);
          } else if (ib == DVM_SK_UN) rv = scalar_unary(sub, x);
          else rv = scalar_arith(sub, x, ib == DVM_SK_BIN ? sget(S, s2) : __uint_as_float(CW(body0 + pc - 1)));
          sset(S, ia, rv);
        } break;
        default:
          err = ST_BAD_CODE;
          pc = body_words;  // stop walking code that cannot be decoded
          break;
      }
    }

    // ---- advance to the next tile ----
    c = cn;
    prog_idx = next_prog_idx;
    tile = next;
    buf ^= 1;
  }
  cp_async_wait<0>();

  if (err && tid == 0) atomicMax(prm.status, err);
  if (use_queue) {
    // the last CTA to finish returns the queue to its resting state (both counters zero)
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      const unsigned done = atomicAdd(&prm.queue[1], 1u);
      if (done == gridDim.x - 1) {
        prm.queue[0] = 0u;
        prm.queue[1] = 0u;
        __threadfence();
      }
    }
  }
#undef DVM_EACH_PAIR
#undef CW
}

}  // namespace dvm
