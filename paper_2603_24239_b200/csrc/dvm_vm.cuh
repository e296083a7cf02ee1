// Device half of the operator compiler: the virtual machine (Sec. 4.3, Algorithm 2)
// as a persistent sm_100a kernel.
//
// One CTA of 256 threads is one "core" of Algorithm 2.  It copies the bytecode
// program(s) from the kernel-parameter block into shared memory once, then loops
// over its tiles; per tile every warp walks the code body, decoding one
// instruction word at a time (a warp-uniform shared-memory read and a uniform
// branch) and executing the tile-level virtual instruction on register-resident
// tile registers.
//
// Tile geometry (chosen per instance by the host's shape tiling):
//   G = 2^lgG threads share one row; a CTA holds 256/G rows per tile.
//   Every thread owns V = 16 element slots of each tile register; slot s maps to
//   column  (t + G*(s / W)) * W + (s % W) - shift  of the tile's column block,
//   t = thread index inside the row group, W = vector width in elements,
//   shift = misalignment of the row segment start, so that a thread's W-slot
//   chunk is a 16-byte aligned vector of the primary operand.
// Tile registers R0..R{NREG-1} hold fp32 values (R0 is the accumulator); S0..S7
// hold one fp32 value per row (reduction results, per-row inputs).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dvm_format.h"

namespace dvm {

constexpr int V = DVM_VM_V;
constexpr int THREADS = DVM_VM_THREADS;

// Device status word values (read back by dvm_last_device_status).
enum { ST_OK = 0, ST_BAD_CODE = 1, ST_TIMEOUT = 2 };

template <int PW>
struct VMParams {
  uint32_t n_programs;
  uint32_t total_tiles;
  uint32_t n_words;      // words used in `words`
  uint32_t use_queue;    // 1: tiles beyond the first are claimed from the work queue
  unsigned int* status;  // device status word
  unsigned int* queue;   // [0] next tile to claim, [1] CTAs finished (both zero between launches)
  uint32_t words[PW];    // [program word offsets][tile prefix sums (n+1)][programs ...]
};

struct TileCtx {
  int t;        // thread index within the row group
  int lgG;
  int W, lgW;
  int shift;
  int ncols;    // valid columns of this thread's row inside the column block (0: nothing to do)
  uint32_t vmask;  // bit s set: slot s holds a valid element
  long long i0, i1, i2;  // row coordinates over the collapsed outer dims
  long long col0;
  bool outer;
};

template <int NREG, class F>
__device__ __forceinline__ void with_reg(float (&R)[NREG][V], int k, F&& f) {
  switch (k) {
    case 0: f(R[0]); break;
    case 1: f(R[1]); break;
    case 2: f(R[2]); break;
    case 3: f(R[3]); break;
    default:
      if constexpr (NREG > 4) {
        switch (k) {
          case 4: f(R[4]); break;
          case 5: f(R[5]); break;
          case 6: f(R[6]); break;
          default: f(R[7]); break;
        }
      }
      break;
  }
}

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

__device__ __forceinline__ float arith(int op, float a, float b) {
  switch (op) {
    case DVM_A_ADD: return a + b;
    case DVM_A_SUB: return a - b;
    case DVM_A_RSUB: return b - a;
    case DVM_A_MUL: return a * b;
    case DVM_A_DIV: return a / b;
    case DVM_A_RDIV: return b / a;
    case DVM_A_MIN: return a < b ? a : b;
    default: return a > b ? a : b;
  }
}

__device__ __forceinline__ float round_bf16(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

__device__ __forceinline__ float unary(int op, float x) {
  switch (op) {
    case DVM_U_EXP: return expf(x);
    case DVM_U_SQRT: return sqrtf(x);
    case DVM_U_RSQRT: return 1.0f / sqrtf(x);
    case DVM_U_ABS: return fabsf(x);
    case DVM_U_LOG: return logf(x);
    case DVM_U_ERF: return erff(x);
    case DVM_U_SIGMOID: return 1.0f / (1.0f + expf(-x));
    case DVM_U_NEG: return -x;
    case DVM_U_RECIP: return 1.0f / x;
    case DVM_U_FLOOR: return floorf(x);
    case DVM_U_ROUND: return rintf(x);
    case DVM_U_TANH: return tanhf(x);
    default: return round_bf16(x);
  }
}

// Column (relative to the column block) of the first slot of chunk j.
__device__ __forceinline__ int chunk_col(const TileCtx& c, int j) {
  return ((c.t + (j << c.lgG)) << c.lgW) - c.shift;
}

// ---- tile load: vector path straight into the destination register ---------------------------
// Raw element bits are written: fp32 as is, bf16 packed two per word (slots 2i, 2i+1 in word i);
// a later CVT instruction widens bf16 in place.  Chunks that straddle the row boundary or are not
// 16-byte aligned are flagged in slow_mask and fetched element-wise by ldg_slow.
template <int W, bool BF16>
__device__ __forceinline__ void ldg_fast(float (&r)[V], const char* p, const TileCtx& c, uint32_t& slow_mask) {
  constexpr int ES = BF16 ? 2 : 4;
#pragma unroll
  for (int i = 0; i < V; ++i) r[i] = 0.f;
  if constexpr (W == 1) {
#pragma unroll
    for (int s = 0; s < V; ++s) {
      int col = c.t + (s << c.lgG);
      if (col < c.ncols) {
        if constexpr (BF16) {
          uint32_t h = *reinterpret_cast<const unsigned short*>(p + (long long)col * ES);
          uint32_t w = __float_as_uint(r[s >> 1]) | (h << (16 * (s & 1)));
          r[s >> 1] = __uint_as_float(w);
        } else {
          r[s] = *reinterpret_cast<const float*>(p + (long long)col * ES);
        }
      }
    }
  } else {
    constexpr int NCH = V / W;
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      int c0 = chunk_col(c, j);
      const char* q = p + (long long)c0 * ES;
      bool full = (c0 >= 0) && (c0 + W <= c.ncols);
      bool al = (reinterpret_cast<uintptr_t>(q) & 15) == 0;
      if (full && al) {
        if constexpr (BF16) {  // W == 8: one 16-byte vector
          uint4 v = *reinterpret_cast<const uint4*>(q);
          r[4 * j + 0] = __uint_as_float(v.x);
          r[4 * j + 1] = __uint_as_float(v.y);
          r[4 * j + 2] = __uint_as_float(v.z);
          r[4 * j + 3] = __uint_as_float(v.w);
        } else {
#pragma unroll
          for (int h = 0; h < W / 4; ++h) {
            float4 v = *reinterpret_cast<const float4*>(q + 16 * h);
            r[W * j + 4 * h + 0] = v.x;
            r[W * j + 4 * h + 1] = v.y;
            r[W * j + 4 * h + 2] = v.z;
            r[W * j + 4 * h + 3] = v.w;
          }
        }
      } else if (c0 + W > 0 && c0 < c.ncols) {
        slow_mask |= 1u << j;
      }
    }
  }
}

// Element-wise fetch of the chunks flagged in slow_mask into tmp (same raw layout).
template <int W, bool BF16>
__device__ __noinline__ void ldg_slow(float (&tmp)[V], const char* p, const TileCtx& c, uint32_t slow_mask) {
  constexpr int ES = BF16 ? 2 : 4;
  constexpr int NCH = V / W;
#pragma unroll
  for (int i = 0; i < V; ++i) tmp[i] = 0.f;
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    if (!((slow_mask >> j) & 1)) continue;
    int c0 = chunk_col(c, j);
#pragma unroll
    for (int e = 0; e < W; ++e) {
      int col = c0 + e;
      int s = W * j + e;
      if (col >= 0 && col < c.ncols) {
        if constexpr (BF16) {
          uint32_t h = *reinterpret_cast<const unsigned short*>(p + (long long)col * ES);
          uint32_t w = __float_as_uint(tmp[s >> 1]) | (h << (16 * (s & 1)));
          tmp[s >> 1] = __uint_as_float(w);
        } else {
          tmp[s] = *reinterpret_cast<const float*>(p + (long long)col * ES);
        }
      }
    }
  }
}

template <int W, bool BF16>
__device__ __forceinline__ void merge_slow(float (&r)[V], const float (&tmp)[V], uint32_t slow_mask) {
  constexpr int NCH = V / W;
  constexpr int WPC = BF16 ? W / 2 : W;  // raw words per chunk
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    bool take = (slow_mask >> j) & 1;
#pragma unroll
    for (int i = 0; i < WPC; ++i) r[WPC * j + i] = take ? tmp[WPC * j + i] : r[WPC * j + i];
  }
}

// ---- tile store from the accumulator -------------------------------------------------------------
template <int W, bool BF16>
__device__ __forceinline__ void stg_tile(const float (&a)[V], char* p, const TileCtx& c) {
  constexpr int ES = BF16 ? 2 : 4;
  if constexpr (W == 1) {
#pragma unroll
    for (int s = 0; s < V; ++s) {
      int col = c.t + (s << c.lgG);
      if (col < c.ncols) {
        if constexpr (BF16) *reinterpret_cast<__nv_bfloat16*>(p + (long long)col * ES) = __float2bfloat16_rn(a[s]);
        else *reinterpret_cast<float*>(p + (long long)col * ES) = a[s];
      }
    }
  } else {
    constexpr int NCH = V / W;
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      int c0 = chunk_col(c, j);
      char* q = p + (long long)c0 * ES;
      bool full = (c0 >= 0) && (c0 + W <= c.ncols);
      bool al = (reinterpret_cast<uintptr_t>(q) & 15) == 0;
      if (full && al) {
        if constexpr (BF16) {
          uint4 v;
          __nv_bfloat162 b0 = __floats2bfloat162_rn(a[8 * j + 0], a[8 * j + 1]);
          __nv_bfloat162 b1 = __floats2bfloat162_rn(a[8 * j + 2], a[8 * j + 3]);
          __nv_bfloat162 b2 = __floats2bfloat162_rn(a[8 * j + 4], a[8 * j + 5]);
          __nv_bfloat162 b3 = __floats2bfloat162_rn(a[8 * j + 6], a[8 * j + 7]);
          v.x = *reinterpret_cast<uint32_t*>(&b0);
          v.y = *reinterpret_cast<uint32_t*>(&b1);
          v.z = *reinterpret_cast<uint32_t*>(&b2);
          v.w = *reinterpret_cast<uint32_t*>(&b3);
          *reinterpret_cast<uint4*>(q) = v;
        } else {
#pragma unroll
          for (int h = 0; h < W / 4; ++h)
            *reinterpret_cast<float4*>(q + 16 * h) =
                make_float4(a[W * j + 4 * h], a[W * j + 4 * h + 1], a[W * j + 4 * h + 2], a[W * j + 4 * h + 3]);
        }
      } else if (c0 + W > 0 && c0 < c.ncols) {
#pragma unroll
        for (int e = 0; e < W; ++e) {
          int col = c0 + e;
          if (col >= 0 && col < c.ncols) {
            if constexpr (BF16)
              *reinterpret_cast<__nv_bfloat16*>(p + (long long)col * ES) = __float2bfloat16_rn(a[W * j + e]);
            else
              *reinterpret_cast<float*>(p + (long long)col * ES) = a[W * j + e];
          }
        }
      }
    }
  }
}

// bf16 raw words -> fp32 values, in place (descending so that no raw word is overwritten early).
__device__ __forceinline__ void widen_bf16(float (&r)[V]) {
#pragma unroll
  for (int i = V / 2 - 1; i >= 0; --i) {
    uint32_t w = __float_as_uint(r[i]);
    r[2 * i + 1] = __uint_as_float(w & 0xffff0000u);
    r[2 * i] = __uint_as_float(w << 16);
  }
}

struct OperandAddr {
  char* ptr;    // address of element (row, col0) -- or of the row's single value for col_stride 0
  int dtype;
};

__device__ __forceinline__ OperandAddr operand_addr(const uint32_t* prog, const uint32_t* opd_table, int b,
                                                    const TileCtx& c) {
  const uint32_t* d = opd_table + b * DVM_OPD_WORDS;
  uint32_t info = d[DVM_OPD_INFO];
  int slot = info & 0xff;
  int dt = (info >> 8) & 0xff;
  int cs = (info >> 16) & 0xff;
  const uint32_t* tp = prog + DVM_HDR_WORDS + 2 * slot;
  unsigned long long base = (unsigned long long)tp[0] | ((unsigned long long)tp[1] << 32);
  long long s0 = (long long)((unsigned long long)d[DVM_OPD_STRIDE0] | ((unsigned long long)d[DVM_OPD_STRIDE0 + 1] << 32));
  long long off = c.i0 * s0;
  if (c.outer) {
    long long s1 = (long long)((unsigned long long)d[DVM_OPD_STRIDE1] | ((unsigned long long)d[DVM_OPD_STRIDE1 + 1] << 32));
    long long s2 = (long long)((unsigned long long)d[DVM_OPD_STRIDE2] | ((unsigned long long)d[DVM_OPD_STRIDE2 + 1] << 32));
    off += c.i1 * s1 + c.i2 * s2;
  }
  if (cs) off += c.col0;
  OperandAddr a;
  a.ptr = reinterpret_cast<char*>(base) + off * (dt == DVM_DT_BF16 ? 2 : 4);
  a.dtype = dt;
  return a;
}

template <int NREG, int PW>
__global__ void __launch_bounds__(THREADS, (NREG <= 4 ? 2 : 1))
dvm_vm_kernel(const __grid_constant__ VMParams<PW> prm) {
  extern __shared__ __align__(16) uint32_t s_code[];
  __shared__ float s_red[2][THREADS / 32];
  __shared__ uint32_t s_next[2];

  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  for (uint32_t i = tid; i < prm.n_words; i += THREADS) s_code[i] = prm.words[i];
  __syncthreads();

  const uint32_t n_prog = prm.n_programs;
  const uint32_t* tile_base = s_code + n_prog;
  float R[NREG][V];
  float S[DVM_MAX_SREGS];
#pragma unroll
  for (int i = 0; i < DVM_MAX_SREGS; ++i) S[i] = 0.f;
#pragma unroll
  for (int k = 0; k < NREG; ++k)
#pragma unroll
    for (int i = 0; i < V; ++i) R[k][i] = 0.f;

  uint32_t prog_idx = 0;
  uint32_t tile = blockIdx.x;
  uint32_t iter = 0;
  int red_par = 0;
  unsigned err = 0;

  while (tile < prm.total_tiles) {
    if (prm.use_queue && tid == 0) s_next[iter & 1] = atomicAdd(&prm.queue[0], 1u) + gridDim.x;

    // ---- locate the program of this tile (stacked launches); tiles are claimed in increasing order ----
    while (prog_idx + 1 < n_prog && tile >= tile_base[prog_idx + 1]) ++prog_idx;
    const uint32_t* prog = s_code + s_code[prog_idx];
    const uint32_t counts = prog[DVM_H_COUNTS];
    const uint32_t n_tensors = counts & 0xff, n_opd = (counts >> 16) & 0xff;
    const uint32_t* opd_table = prog + DVM_HDR_WORDS + 2 * n_tensors;
    const uint32_t* body = opd_table + n_opd * DVM_OPD_WORDS;
    const uint32_t body_words = prog[DVM_H_CODE_WORDS];
    const uint32_t geom = prog[DVM_H_GEOM];

    TileCtx c;
    c.lgG = geom & 0xff;
    c.W = (geom >> 8) & 0xff;
    c.lgW = c.W == 8 ? 3 : (c.W == 4 ? 2 : 0);
    const uint32_t flags = geom >> 24;
    c.outer = (flags & DVM_F_OUTER_DIMS) != 0;
    const int G = 1 << c.lgG;
    c.t = tid & (G - 1);
    const int g = tid >> c.lgG;
    const uint32_t local_tile = tile - tile_base[prog_idx];
    const uint32_t CB = prog[DVM_H_COL_BLOCKS];
    uint32_t rb = local_tile, cb = 0;
    if (CB > 1) { rb = local_tile / CB; cb = local_tile - rb * CB; }
    const long long rows = (long long)((unsigned long long)prog[DVM_H_ROWS_LO] | ((unsigned long long)prog[DVM_H_ROWS_HI] << 32));
    const long long row = (long long)rb * (THREADS >> c.lgG) + g;
    const uint32_t ctile = prog[DVM_H_COL_TILE];
    c.col0 = (long long)cb * ctile;
    {
      long long cend = (row == rows - 1) ? (long long)prog[DVM_H_LAST_ROW_COLS] : (long long)prog[DVM_H_COLS];
      long long nc = cend - c.col0;
      if (nc > (long long)ctile) nc = ctile;
      if (nc < 0 || row >= rows) nc = 0;
      c.ncols = (int)nc;
    }
    c.i0 = row < rows ? row : 0;
    c.i1 = c.i2 = 0;
    if (c.outer) {
      unsigned long long n0 = prog[DVM_H_OUTER0], n1 = prog[DVM_H_OUTER1];
      unsigned long long q = (unsigned long long)c.i0 / n0;
      c.i0 = (long long)((unsigned long long)c.i0 - q * n0);
      unsigned long long q2 = q / n1;
      c.i1 = (long long)(q - q2 * n1);
      c.i2 = (long long)q2;
    }
    c.shift = 0;
    if (!(flags & DVM_F_ALIGNED) && c.W > 1) {
      const uint32_t pr = prog[DVM_H_PRIMARY];
      if (pr != 0xffffffffu) {
        OperandAddr pa = operand_addr(prog, opd_table, (int)pr, c);
        unsigned long long e = reinterpret_cast<unsigned long long>(pa.ptr) >> (pa.dtype == DVM_DT_BF16 ? 1 : 2);
        c.shift = (int)(e & (unsigned long long)(c.W - 1));
      }
    }
    {
      uint32_t m = 0;
#pragma unroll
      for (int s = 0; s < V; ++s) {
        int col = ((c.t + ((s >> c.lgW) << c.lgG)) << c.lgW) + (s & (c.W - 1)) - c.shift;
        if (col >= 0 && col < c.ncols) m |= 1u << s;
      }
      c.vmask = m;
    }

    // ---- Algorithm 2, inner loop: walk the code body ----
    float (&A)[V] = R[0];
    uint32_t pc = 0;
    while (pc < body_words) {
      const uint32_t w0 = body[pc];
      const uint32_t op = DVM_INSN_OP(w0);
      const int ia = DVM_INSN_A(w0), ib = DVM_INSN_B(w0);
      const uint32_t len = DVM_INSN_LEN(w0);
      if (op >= DVM_OP_BIN && op < DVM_OP_BIN + 8 * DVM_A_NBIN) {
        const int ar = (op - DVM_OP_BIN) >> 3, k = (op - DVM_OP_BIN) & 7;
        switch (ar) {
#define DVM_BIN_CASE(AR, EXPR)                                   \
  case AR:                                                       \
    with_reg<NREG>(R, k, [&](float (&r)[V]) {                    \
      _Pragma("unroll") for (int i = 0; i < V; ++i) {            \
        const float x = A[i], y = r[i];                          \
        A[i] = (EXPR);                                           \
      }                                                          \
    });                                                          \
    break;
          DVM_BIN_CASE(DVM_A_ADD, x + y)
          DVM_BIN_CASE(DVM_A_SUB, x - y)
          DVM_BIN_CASE(DVM_A_RSUB, y - x)
          DVM_BIN_CASE(DVM_A_MUL, x * y)
          DVM_BIN_CASE(DVM_A_DIV, x / y)
          DVM_BIN_CASE(DVM_A_RDIV, y / x)
          DVM_BIN_CASE(DVM_A_MIN, x < y ? x : y)
          DVM_BIN_CASE(DVM_A_MAX, x > y ? x : y)
#undef DVM_BIN_CASE
        }
      } else if (op >= DVM_OP_BINS && op < DVM_OP_BINS + DVM_A_NBIN) {
        const float y = sget(S, ia);
        switch (op - DVM_OP_BINS) {
#define DVM_BINS_CASE(AR, EXPR)                                                                  \
  case AR:                                                                                       \
    _Pragma("unroll") for (int i = 0; i < V; ++i) { const float x = A[i]; A[i] = (EXPR); }       \
    break;
          DVM_BINS_CASE(DVM_A_ADD, x + y)
          DVM_BINS_CASE(DVM_A_SUB, x - y)
          DVM_BINS_CASE(DVM_A_RSUB, y - x)
          DVM_BINS_CASE(DVM_A_MUL, x * y)
          DVM_BINS_CASE(DVM_A_DIV, x / y)
          DVM_BINS_CASE(DVM_A_RDIV, y / x)
          DVM_BINS_CASE(DVM_A_MIN, x < y ? x : y)
          DVM_BINS_CASE(DVM_A_MAX, x > y ? x : y)
        }
      } else if (op >= DVM_OP_BINI && op < DVM_OP_BINI + DVM_A_NBIN) {
        const float y = __uint_as_float(body[pc + 1]);
        switch (op - DVM_OP_BINI) {
          DVM_BINS_CASE(DVM_A_ADD, x + y)
          DVM_BINS_CASE(DVM_A_SUB, x - y)
          DVM_BINS_CASE(DVM_A_RSUB, y - x)
          DVM_BINS_CASE(DVM_A_MUL, x * y)
          DVM_BINS_CASE(DVM_A_DIV, x / y)
          DVM_BINS_CASE(DVM_A_RDIV, y / x)
          DVM_BINS_CASE(DVM_A_MIN, x < y ? x : y)
          DVM_BINS_CASE(DVM_A_MAX, x > y ? x : y)
#undef DVM_BINS_CASE
        }
      } else if (op >= DVM_OP_UN && op < DVM_OP_UN + DVM_U_NUN) {
        switch (op - DVM_OP_UN) {
#define DVM_UN_CASE(U, EXPR)                                                                     \
  case U:                                                                                        \
    _Pragma("unroll") for (int i = 0; i < V; ++i) { const float x = A[i]; A[i] = (EXPR); }       \
    break;
          DVM_UN_CASE(DVM_U_EXP, expf(x))
          DVM_UN_CASE(DVM_U_SQRT, sqrtf(x))
          DVM_UN_CASE(DVM_U_RSQRT, 1.0f / sqrtf(x))
          DVM_UN_CASE(DVM_U_ABS, fabsf(x))
          DVM_UN_CASE(DVM_U_LOG, logf(x))
          DVM_UN_CASE(DVM_U_ERF, erff(x))
          DVM_UN_CASE(DVM_U_SIGMOID, 1.0f / (1.0f + expf(-x)))
          DVM_UN_CASE(DVM_U_NEG, -x)
          DVM_UN_CASE(DVM_U_RECIP, 1.0f / x)
          DVM_UN_CASE(DVM_U_FLOOR, floorf(x))
          DVM_UN_CASE(DVM_U_ROUND, rintf(x))
          DVM_UN_CASE(DVM_U_TANH, tanhf(x))
          DVM_UN_CASE(DVM_U_RND_BF16, round_bf16(x))
#undef DVM_UN_CASE
        }
      } else if (op >= DVM_OP_RED && op < DVM_OP_RED + DVM_R_NRED) {
        // row reduction: thread-local over valid slots, shuffles inside the warp, shared memory across
        // the warps of a row group (Table 1, Sum / Max / Min with N = 1)
        const int rop = op - DVM_OP_RED;
        const float ident = rop == DVM_R_SUM ? 0.f : (rop == DVM_R_MAX ? -INFINITY : INFINITY);
        float v = ident;
#pragma unroll
        for (int i = 0; i < V; ++i) {
          const float x = ((c.vmask >> i) & 1) ? A[i] : ident;
          v = rop == DVM_R_SUM ? v + x : (rop == DVM_R_MAX ? (x > v ? x : v) : (x < v ? x : v));
        }
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          if (o < G) {
            const float x = __shfl_xor_sync(0xffffffffu, v, o);
            v = rop == DVM_R_SUM ? v + x : (rop == DVM_R_MAX ? (x > v ? x : v) : (x < v ? x : v));
          }
        }
        if (G > 32) {
          if (lane == 0) s_red[red_par][warp] = v;
          __syncthreads();
          const int wpg = G >> 5;          // warps per row group
          const int w0i = (warp / wpg) * wpg;
          float acc = ident;
          for (int i = 0; i < wpg; ++i) {
            const float x = s_red[red_par][w0i + i];
            acc = rop == DVM_R_SUM ? acc + x : (rop == DVM_R_MAX ? (x > acc ? x : acc) : (x < acc ? x : acc));
          }
          v = acc;
          red_par ^= 1;
        }
        sset(S, ia, v);
      } else {
        switch (op) {
          case DVM_OP_NOP: break;
          case DVM_OP_LDG: {
            const OperandAddr oa = operand_addr(prog, opd_table, ib, c);
            uint32_t slow = 0;
            const int variant = (oa.dtype == DVM_DT_BF16 ? 1 : 0) | (c.W == 8 ? 2 : (c.W == 4 ? 4 : 0));
            with_reg<NREG>(R, ia, [&](float (&r)[V]) {
              switch (variant) {
                case 0: ldg_fast<1, false>(r, oa.ptr, c, slow); break;
                case 1: ldg_fast<1, true>(r, oa.ptr, c, slow); break;
                case 2: ldg_fast<8, false>(r, oa.ptr, c, slow); break;
                case 3: ldg_fast<8, true>(r, oa.ptr, c, slow); break;
                case 4: ldg_fast<4, false>(r, oa.ptr, c, slow); break;
                default: err = ST_BAD_CODE; break;
              }
            });
            if (slow) {
              float tmp[V];
              switch (variant) {
                case 2: ldg_slow<8, false>(tmp, oa.ptr, c, slow); break;
                case 3: ldg_slow<8, true>(tmp, oa.ptr, c, slow); break;
                default: ldg_slow<4, false>(tmp, oa.ptr, c, slow); break;
              }
              with_reg<NREG>(R, ia, [&](float (&r)[V]) {
                switch (variant) {
                  case 2: merge_slow<8, false>(r, tmp, slow); break;
                  case 3: merge_slow<8, true>(r, tmp, slow); break;
                  default: merge_slow<4, false>(r, tmp, slow); break;
                }
              });
            }
          } break;
          case DVM_OP_CVT:
            if (ib == DVM_DT_BF16) with_reg<NREG>(R, ia, [&](float (&r)[V]) { widen_bf16(r); });
            break;
          case DVM_OP_STG: {
            const OperandAddr oa = operand_addr(prog, opd_table, ib, c);
            const int variant = (oa.dtype == DVM_DT_BF16 ? 1 : 0) | (c.W == 8 ? 2 : (c.W == 4 ? 4 : 0));
            switch (variant) {
              case 0: stg_tile<1, false>(A, oa.ptr, c); break;
              case 1: stg_tile<1, true>(A, oa.ptr, c); break;
              case 2: stg_tile<8, false>(A, oa.ptr, c); break;
              case 3: stg_tile<8, true>(A, oa.ptr, c); break;
              case 4: stg_tile<4, false>(A, oa.ptr, c); break;
              default: err = ST_BAD_CODE; break;
            }
          } break;
          case DVM_OP_LDS: {
            const OperandAddr oa = operand_addr(prog, opd_table, ib, c);
            float v = 0.f;
            if (c.ncols > 0) {
              if (oa.dtype == DVM_DT_BF16) v = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(oa.ptr));
              else v = *reinterpret_cast<const float*>(oa.ptr);
            }
            sset(S, ia, v);
          } break;
          case DVM_OP_STS: {
            const OperandAddr oa = operand_addr(prog, opd_table, ib, c);
            const float v = sget(S, ia);
            if (c.ncols > 0 && c.t == 0 && c.col0 == 0) {
              if (oa.dtype == DVM_DT_BF16) *reinterpret_cast<__nv_bfloat16*>(oa.ptr) = __float2bfloat16_rn(v);
              else *reinterpret_cast<float*>(oa.ptr) = v;
            }
          } break;
          case DVM_OP_MOV:
            if (ia == 0) {
              with_reg<NREG>(R, ib, [&](float (&r)[V]) {
#pragma unroll
                for (int i = 0; i < V; ++i) A[i] = r[i];
              });
            } else {
              with_reg<NREG>(R, ia, [&](float (&r)[V]) {
#pragma unroll
                for (int i = 0; i < V; ++i) r[i] = A[i];
              });
            }
            break;
          case DVM_OP_BCS: {
            const float v = sget(S, ia);
#pragma unroll
            for (int i = 0; i < V; ++i) A[i] = v;
          } break;
          case DVM_OP_SOP: {
            const uint32_t w1 = body[pc + 1];
            const int sub = w1 & 0xff, s1 = (w1 >> 8) & 0xff, s2 = (w1 >> 16) & 0xff;
            const float x = sget(S, s1);
            float rv;
            if (ib == DVM_SK_BIN) rv = arith(sub, x, sget(S, s2));
            else if (ib == DVM_SK_BINI) rv = arith(sub, x, __uint_as_float(body[pc + 2]));
            else rv = unary(sub, x);
            sset(S, ia, rv);
          } break;
          default:
            err = ST_BAD_CODE;
            break;
        }
      }
      pc += len ? len : 1;  // Insn_Len; the host verifier rejects len == 0, this only bounds the walk
    }

    ++iter;
    if (prm.use_queue) {
      __syncthreads();
      tile = s_next[(iter - 1) & 1];
    } else {
      tile += gridDim.x;
    }
  }

  if (err && tid == 0) atomicMax(prm.status, err);
  if (prm.use_queue) {
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
}

}  // namespace dvm
