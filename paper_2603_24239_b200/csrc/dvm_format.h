// Bytecode program format of the device-side virtual machine (host + device).
//
// The paper fixes only the parts list (Sec. 4.2 "Bytecode encoding"): a code
// header {KernelType, CodeSize, total number of tiles} and a code body with one
// bytecode per operation {instruction id, bytecode length, source / destination
// tile operands, compute size, extras}.  Field widths and ids are this
// library's own.  Everything is 32-bit little-endian words.
//
//   [ header : DVM_HDR_WORDS words ]
//   [ tensor table : 2 words per tensor slot (device pointer, patched at launch) ]
//   [ operand table : DVM_OPD_WORDS words per global-memory operand ]
//   [ local register table : one word per local register: its unit offset inside a tile slot ]
//   [ code body : CodeSize words, instructions of 1..3 words ]
//
// Unlike the paper's bytecode, a memory instruction does not carry an address:
// it names an operand descriptor, which names a tensor slot; the launch call
// supplies the pointers.  The tile id an instruction needs (Algorithm 2) is the
// interpreter's loop variable.
#pragma once
#include <stdint.h>

#define DVM_MAGIC 0x314D5644u /* "DVM1" */

enum {
  DVM_KERNEL_VEC = 1,     // meta-kernel of vector operations
  DVM_KERNEL_MATMUL = 2,  // meta-kernel: matmul instruction + fused epilogue
  DVM_KERNEL_STACKED = 3  // several meta-kernels in one launch (built at launch time)
};

// ---- header word indices ----
enum {
  DVM_H_MAGIC = 0,
  DVM_H_KERNEL_TYPE = 1,
  DVM_H_CODE_WORDS = 2,   // CodeSize: body length in words
  DVM_H_N_TILES = 3,      // total number of tiles
  DVM_H_TOTAL_WORDS = 4,  // header + tables + body
  DVM_H_COUNTS = 5,       // n_tensors | n_inputs << 8 | n_operands << 16 | n_outputs << 24
  DVM_H_GEOM = 6,         // log2G | W << 8 | local registers << 16 | flags << 24
  DVM_H_COLS = 7,         // C: columns of the dominant (collapsed) shape
  DVM_H_ROWS_LO = 8,      // R: rows of the dominant shape (64 bit)
  DVM_H_ROWS_HI = 9,
  DVM_H_COL_BLOCKS = 10,  // number of column blocks per row group
  DVM_H_COL_TILE = 11,    // columns per column block
  DVM_H_OUTER0 = 12,      // sizes of the (up to 3) collapsed outer dims, innermost first
  DVM_H_OUTER1 = 13,
  DVM_H_OUTER2 = 14,
  DVM_H_LAST_ROW_COLS = 15,  // valid columns of the last row (flat programs), else C
  DVM_H_PRIMARY = 16,        // operand whose row starts define the vector alignment, or 0xffffffff
  DVM_H_LOCAL = 17,          // n_in_regs | n_tmp_regs << 8 | n_scalar_slots << 16 | V << 24 (elements per thread: 16 or 32)
  DVM_H_LOAD_WORDS = 18,     // length of the load section (words) at the start of the code body
  DVM_H_LOCAL2 = 19,         // unit offset of the per-row scalar slots | units of one tile slot << 16
  DVM_HDR_WORDS = 20
};

// flags in DVM_H_GEOM bits 24..31
enum {
  DVM_F_ALIGNED = 1,    // every row segment of the primary operand starts on a W-element
                        // boundary provided its base pointer is 16-byte aligned
  DVM_F_OUTER_DIMS = 2, // row index must be decomposed over OUTER0..2 for some operand
  DVM_F_FLAT = 4,       // pure elementwise program laid out as a flat range
  DVM_F_PRIMARY_DENSE = 8, // the primary operand is dense: row r starts at element r * C of its tensor
  DVM_F_EXT_ISA = 32,      // the program uses Cmp / Select / Pow / IsFinite: it needs the extended interpreter variant
  DVM_F_VIEWS = 64,        // a gathered input or a tile stored into a strided view: it needs the views variant
  DVM_F_ONE_SLOT = 128,    // hint to dvm_launch: two tile slots leave room for one CTA per SM, one slot for two -- run the
                           // program with a single slot (no prefetch inside a CTA; the SM's other CTA covers the loads)
  DVM_F_LOADS_BY_ROW = 16  // some load is issued per row (row-by-row images, per-row scalars); otherwise
                           // thread 0 alone issues every copy of a tile
};

// ---- local register table: one word per local register:
//      unit offset inside a tile slot | mode << 16 | (tensor address & 15) << 20 (set at launch) | operand << 24 ----
enum {
  DVM_LM_PRIVATE = 0,  // temporary: thread-private fp32 vectors, vector q of thread tid at (q * 256 + tid) * 16
  DVM_LM_BLOCK = 1,    // input whose tile is one contiguous byte range of global memory: one bulk copy per tile
  DVM_LM_ROWS = 2,     // input copied row by row (one bulk copy per row): row images DVM_ROW_PITCH(...) apart
  DVM_LM_BCAST = 3,    // row-vector input, the same for every row and tile: one row image per slot, loaded once per
                       // slot and program
  DVM_LM_BCAST_TILE = 4, // the same with several column blocks: the image holds the tile's column block, loaded with every tile
  DVM_LM_GATHER = 5,   // input whose columns are not adjacent in memory (Table 1, ViewLoad): every thread fetches its own
                       // elements, widened to fp32, into the thread-private layout of a temporary (extended variant)
  DVM_LM_TRANSPOSED = 6 // such an input whose ROWS are adjacent in memory (a transposed matrix): the tile's part of every column
                       // is one contiguous strip -- one bulk copy per column into strip images DVM_STRIP_PITCH apart; a thread
                       // reads its row's element of each of its columns from the strips (raw element type; the instructions
                       // that read the register say fp32, as for a gathered one)
};
// bytes between the strip images of a TRANSPOSED register (R rows of the tile; alignment slack on both sides)
#define DVM_STRIP_PITCH(R, es) ((uint32_t)(R) * (uint32_t)(es) + 32u)
// bytes between the row images of a ROWS register (room for the 16-byte alignment slack on both sides)
#define DVM_ROW_PITCH(G, V, es) ((uint32_t)(G) * (uint32_t)(V) * (uint32_t)(es) + 32u)

// ---- operand descriptor ----
enum {
  DVM_OPD_INFO = 0,      // tensor slot | dtype << 8 | col_stride << 16 | primary << 24 | dense << 25 | combine << 26
                         // (combine, outputs only: 0 plain store; 1 sum, 2 max, 3 min: every tile combines its rows into
                         //  the fp32 result with atomic operations -- a reduction over an axis the tiles walk along)
                         // (dense: element (row, col) sits at flat offset row * C + col)
  DVM_OPD_COLSTRIDE = 1, // element stride between the columns of a tile-class operand: 1, or a view's (then gathered / scattered)
  DVM_OPD_STRIDE0 = 2,   // int64 element stride of outer dim 0 (lo, hi)
  DVM_OPD_STRIDE1 = 4,
  DVM_OPD_STRIDE2 = 6,
  DVM_OPD_FILL = 7,      // combined output: its element count (the launch pre-fills it with the operation's identity);
                         // the word is the high half of stride 2, always 0 otherwise (strides stay below 2^32)
  DVM_OPD_WORDS = 8
};

enum { DVM_DT_F32 = 0, DVM_DT_BF16 = 1,
       DVM_DT_U8 = 2, DVM_DT_I32 = 3 };  // outputs only: the stored value is the fp32 register converted toward zero (Table 1, Cast)
// log2 of an element's bytes: bf16 1, fp32 / i32 2, u8 0
#define DVM_DT_LG_ES(dt) ((dt) == DVM_DT_BF16 ? 1 : ((dt) == DVM_DT_U8 ? 0 : 2))

// ---- limits ----
#define DVM_VM_THREADS 256       // threads per CTA of the interpreter
#define DVM_VM_VMAX 32           // most elements of a tile register one thread holds (V is 16 or 32)
#define DVM_MAX_LREGS 10         // local tile registers of a program (inputs + temporaries)
#define DVM_MAX_SSLOTS 8         // per-row scalar inputs of a program
#define DVM_LOCAL_UNIT 256       // bytes of one local-memory unit (layout granule)
#define DVM_MAX_LOCAL_UNITS 864  // units a CTA can hold (two tile slots + the spare unit), 216 KB
#define DVM_MAX_SREGS 8          // per-row scalar registers
#define DVM_MAX_TENSORS 16
#define DVM_MAX_OPERANDS 24
#define DVM_MAX_NODES 96
#define DVM_MAX_STACK 256        // programs per stacked launch

// ---- instruction word 0:  op | len << 8 | a << 16 | b << 24 ----
#define DVM_INSN(op, len, a, b) \
  ((uint32_t)(op) | ((uint32_t)(len) << 8) | ((uint32_t)(a) << 16) | ((uint32_t)(b) << 24))
#define DVM_INSN_OP(w) ((w) & 0xffu)
#define DVM_INSN_LEN(w) (((w) >> 8) & 0xfu)
// bits 12..15 of word 0: the phase tag of an instruction of a phased program (see DVM_OP_PHASE); 0 everywhere else
#define DVM_INSN_TAG(w) (((w) >> 12) & 0xfu)
#define DVM_INSN_SET_TAG(w, t) (((w) & ~0xf000u) | ((uint32_t)(t) << 12))
#define DVM_INSN_A(w) (((w) >> 16) & 0xffu)
#define DVM_INSN_B(w) (((w) >> 24) & 0xffu)

// Arithmetic sub-operations (shared numbering for tile and scalar forms).
enum {
  DVM_A_ADD = 0, DVM_A_SUB = 1, DVM_A_RSUB = 2, DVM_A_MUL = 3,
  DVM_A_DIV = 4, DVM_A_RDIV = 5, DVM_A_MIN = 6, DVM_A_MAX = 7,
  DVM_A_NBIN = 8
};
enum {
  DVM_U_EXP = 0, DVM_U_SQRT = 1, DVM_U_RSQRT = 2, DVM_U_ABS = 3, DVM_U_LOG = 4,
  DVM_U_ERF = 5, DVM_U_SIGMOID = 6, DVM_U_NEG = 7, DVM_U_RECIP = 8, DVM_U_FLOOR = 9,
  DVM_U_ROUND = 10, DVM_U_TANH = 11, DVM_U_RND_BF16 = 12,
  DVM_U_ISFINITE = 13,  // Table 1, IsFinite: 1.0 for a finite value, else 0.0 (tile class: extended variant only)
  DVM_U_TRUNC_I32 = 14, // Table 1, Cast to i32: the fraction dropped toward zero, the value kept inside the type's range (fp32 register)
  DVM_U_TRUNC_U8 = 15,  // ... to u8
  DVM_U_NUN = 16
};
enum { DVM_ACT_GELU = 0, DVM_ACT_SILU = 1, DVM_ACT_N = 2 };
// the two-tile-operand class of the extended variant: the comparisons (Table 1, Cmp) and Pow (Table 1)
enum { DVM_C_GT = 0, DVM_C_GE = 1, DVM_C_LT = 2, DVM_C_LE = 3, DVM_C_EQ = 4, DVM_C_NE = 5,
       DVM_C_POW = 6,   // ACC = ACC ^ L[a]
       DVM_C_RPOW = 7,  // ACC = L[a] ^ ACC
       DVM_C_NCMP = 8 };
// SUMSQ (sum of squares of R0, R0 kept) is what the encoder emits for reduce_sum(x * x).
enum { DVM_R_SUM = 0, DVM_R_MAX = 1, DVM_R_MIN = 2, DVM_R_SUMSQ = 3, DVM_R_NRED = 4 };

// Instruction ids.  The code body is [load section][compute section].
// ACC is the register-resident accumulator tile; L[k] are tile registers in local (shared) memory,
// thread-private, k < n_in: input registers, k >= n_in: temporaries; S[k] are per-row scalars.
// A CTA holds two tile slots (complete sets of local registers): the load section of tile i+1 fills one
// slot while tile i is computed in the other; a row-vector input of an aligned program is the same for
// every tile of a thread and is loaded once per slot.
enum {
  DVM_OP_NOP = 0x00,
  DVM_OP_LDG = 0x01,   // [load] a = local register (| 0x80: tile-invariant, loaded once per CTA and program),
                       //        b = operand : async tile load (raw element bits)
  DVM_OP_LDS = 0x02,   // [load] a = scalar slot,    b = operand : async load of one value per row
  DVM_OP_LDA = 0x03,   // a = local register, b = dtype of its content : ACC = widen(L[a])
  DVM_OP_STA = 0x04,   // a = local register                           : L[a] = ACC (fp32)   (Table 1, Copy)
  DVM_OP_LSS = 0x05,   // a = scalar register, b = scalar slot          : S[a] = loaded per-row value
  DVM_OP_STG = 0x06,   // b = operand                                  : narrow ACC and store the tile
  DVM_OP_STS = 0x07,   // a = scalar register, b = operand             : store one value per row
  DVM_OP_BCS = 0x08,   // a = scalar register                          : ACC = broadcast(S[a]) (Table 1, Broadcast)
  DVM_OP_SOP = 0x09,   // per-row scalar arithmetic; a = dst scalar register, b = kind;
                       // len 2: word1 = sub_op | src1 << 8 | src2 << 16 ; len 3: word2 = fp32 immediate
  DVM_OP_PHASE = 0x0a, // Rows longer than a tile (Table 1, Sum / Max / Min over a long axis): the program runs in P phases over
                       // the CB column blocks of a row -- a CTA takes a row through P * CB tiles in order, every tile walks
                       // the same code, and the per-row scalars stay in place between them.  A reduction accumulates over
                       // the blocks of its phase and is complete for the next one (a softmax: the maximum, then the sum of
                       // the exponentials, then the quotient).
                       //   a = 0xff, b = P : first compute instruction of a phased program, nothing at run time
                       //   a = q           : the tiles of phases < q end here
                       // Tag t > 0 (DVM_INSN_TAG) on RED / SOP / STS / STG: the instruction runs in phase t - 1 only;
                       // RED in every block of it (combining with the blocks before), SOP and STS in its last block
                       // (right behind the reductions that complete there), STG in every block.
  DVM_OP_BINI = 0x10,  // 0x10 + arith; len 2, word1 = fp32 immediate  : ACC = ACC op imm     (Adds / Muls)
  DVM_OP_BIN = 0x18,   // 0x18 + arith; a = local register or 0xff (ACC itself), b = dtype : ACC = ACC op L[a]
  DVM_OP_BINS = 0x20,  // 0x20 + arith; a = scalar register            : ACC = ACC op S[a]    (row broadcast)
  DVM_OP_UN = 0x28,    // 0x28 + unary (16)                            : ACC = f(ACC)
  DVM_OP_RED = 0x38,   // 0x38 + reduce (4); a = dst scalar register   : S[a] = reduce(ACC) over the row
  DVM_OP_LD2 = 0x40,   // 0x40 + arith; a = local register x, b = local register y | dtype(x) << 6 | dtype(y) << 7
                       //                                             : ACC = L[x] op L[y]   (fused copy + arithmetic)
  DVM_OP_ACT = 0x48,   // 0x48 + activation: ACC = act(ACC), a self-gating chain of Table 1 operations fused by the encoder
                       //   (pattern-based fusion, Sec. 5.1): 0 GELU  0.5 t (1 + erf(t / sqrt 2)),  1 SiLU  t sigmoid(t);
                       //   fused, the chain needs no temporary for t
  DVM_OP_CMP = 0x50,   // 0x50 + comparison; a = local register or 0xff (ACC itself), b = dtype : ACC = ACC cmp L[a] ? 1 : 0
                       //   (0x56 / 0x57: Pow, ACC = ACC ^ L[a] / L[a] ^ ACC)
  DVM_OP_SEL = 0x58,   // Table 1, Select; a = local register p, b = local register q | dtype(p) << 6 | dtype(q) << 7
                       //   0x58: ACC = ACC != 0 ? L[p] : L[q]     (the condition is in the accumulator)
                       //   0x59: ACC = L[p] != 0 ? L[q] : ACC     (the else-value is in the accumulator)
                       //   0x5a: ACC = L[p] != 0 ? ACC : L[q]     (the then-value is in the accumulator)
                       //   0x5b: ACC = ACC != 0 ? imm1 : imm2     (len 3; pattern-based fusion, Sec. 5.1: a Select between two
                       //         scalar multiples (or offsets) of ONE value x is x times (plus) the selected scalar --
                       //         no temporaries for the two candidates, bit-identical results)
  DVM_OP_LAST = 0x60   // every arithmetic class starts at a multiple of 8: the low 3 bits are the operation
};
#define DVM_REG_ACC 0xff
#define DVM_MAX_PHASES 8
// phases of a phased program, from the first word of its compute section; 0: the program is not phased
#define DVM_PHASES_OF(w0) ((DVM_INSN_OP(w0) == DVM_OP_PHASE && DVM_INSN_A(w0) == 0xffu) ? DVM_INSN_B(w0) : 0u)
// DVM_SK_FMAU: S[a] = unary(S[src] * imm0 + imm1); len 4: word1 = unary (0xff: none) | src << 8, word2 = imm0, word3 = imm1
enum { DVM_SK_BIN = 0, DVM_SK_BINI = 1, DVM_SK_UN = 2, DVM_SK_FMAU = 3 };

// ---- matmul meta-kernel (DVM_KERNEL_MATMUL): matmul instruction + interpreted epilogue ----
//   [ header ][ tensor table ][ matmul extension : DVM_MM_WORDS ][ operand table ][ epilogue code ]
// Header fields reused: N_TILES = row blocks x column blocks of the output, COLS = N, ROWS_LO = M.
// The epilogue is accumulator code over one chunk of DVM_MM_CHUNK output columns of one output row
// per thread.  Register operands of LDA / BIN / STA name
//   r <  NB            : the fp32 result of matmul r (tensor memory),
//   NB <= r < NB + n_tmp : a temporary (shared memory),
//   0x80 | k           : global operand k of the operand table (an extra [M,N] / [1,N] / [M,1] input),
//   0xff               : the accumulator itself.
// STG names an operand of the operand table (an output, row-major [M,N]).
enum {
  DVM_MM_M = 0, DVM_MM_N = 1, DVM_MM_K = 2,
  DVM_MM_NB = 3,        // number of B matrices sharing A (1 or 2)
  DVM_MM_TILE_N = 4,    // output columns per tile: 128 (NB = 2) or 256 (NB = 1)
  DVM_MM_SLOTS = 5,     // tensor slot of A | slot of B0 << 8 | slot of B1 << 16
  DVM_MM_NTMP = 6,      // epilogue temporaries
  DVM_MM_MBLOCKS = 7, DVM_MM_NBLOCKS = 8, DVM_MM_KBLOCKS = 9,
  DVM_MM_WORDS = 10
};
#define DVM_MM_BLOCK_M 128   // output rows per tile (one UMMA M)
#define DVM_MM_BLOCK_K 64    // K elements per pipeline stage (one 128-byte swizzle row of bf16)
#define DVM_MM_CHUNK 32      // output columns an epilogue thread holds at a time
#define DVM_MM_MAX_TMP 2
#define DVM_MM_MAX_WORDS 320 // whole matmul program (header, tables, code) in the kernel-parameter block
