// Linked code of the lean interpreter.
//
// dvm_launch places a program in the kernel-parameter block.  For the lean interpreter it also LINKS the
// compute section: every bytecode becomes one record of four words whose fields are ready to use -- handler
// id, byte offsets of local registers inside a tile slot, layout mode and element size of the operand,
// immediates -- so that the device decodes nothing per tile (Sec. 4.3: decode is kept off the execution
// path).  The records replace the compute section in the placed copy; the load section, the header and the
// tables stay as encoded.  Records are private to the library: they never leave dvm_launch.
//
// The linker also rewrites and fuses what the encoder emits separately:
//   ACC op imm / ACC op S[a] for add, sub, rsub, mul, div            -> one multiply-add form  ACC = ACC * m + c
//   multiply by an immediate, then add an immediate                  -> one multiply-add
//   RED followed by a scalar multiply-add(-unary) of its result      -> one reduction with a post-operation
//   ACC = ACC - S[a] followed by exp                                 -> one EXPS
//   ACC = L[x] op L[y] followed by a multiplication by an immediate  -> one LD2 with a post-multiplier
//   ACC = ACC * S[a] followed by ACC = ACC * L[y]                    -> one BIN with a pre-multiplier
// and picks the one-piece exponential (EXPS / exp / sigmoid with the `fast` bit) when every output of the
// program is bf16.
#pragma once
#include <stdint.h>

#include "dvm_format.h"

enum {
  DVM_LK_END = 0,
  // the records of the bf16 sweeps first (DVM_LK_HOT_LAST closes the set: the interpreter tests them as a range)
  DVM_LK_LD2_BF16,                                       // ACC = L[x] op L[y] (* w3 when b) sub = add / sub / rsub / mul, w1, w2 = operand words
  DVM_LK_BIN_BF16,                                       // ACC = ACC op L[y]          sub = arith, w1 = operand word; b = 1 + s: ACC * S[s] * L[y]
  DVM_LK_FMA,                                            // ACC = ACC * m + c          m = sub & 1 ? S[a] : w1 (sub & 4: its reciprocal),
                                                         //                            c = sub & 2 ? S[b] : w2 (sub & 8: negated)
  DVM_LK_EXPS,                                           // ACC = exp(ACC - S[a])      sub = 1: one-piece exponential
  DVM_LK_RED,                                            // S[a] = reduce(ACC); b = 1: S[a] = unary(S[a] * w2 + w3), w1 = unary or 0xff
  DVM_LK_STG,                                            // store ACC: a = log2(element size), w1 | w2 << 32 = tensor address
  DVM_LK_LDA_BF16,                                       // ACC = L[x]                 w1 = operand word
  DVM_LK_HOT_LAST = DVM_LK_LDA_BF16,
  DVM_LK_LDA_F32, DVM_LK_LDA_PRIV,                       // ACC = L[x] (fp32 image, private temporary)
  DVM_LK_BIN_F32, DVM_LK_BIN_PRIV,                       // ACC = ACC op L[y] (as DVM_LK_BIN_BF16)
  DVM_LK_BIN_ACC,                                        // ACC = ACC op ACC           sub = arith
  DVM_LK_BINI,                                           // ACC = ACC op imm           sub = rdiv / min / max, w1 = imm
  DVM_LK_BINS,                                           // ACC = ACC op S[a]          sub = rdiv / min / max
  DVM_LK_ACT,                                            // ACC = act(ACC)             sub = DVM_ACT_* (HEAVY variants)
  DVM_LK_UN,                                             // ACC = f(ACC)               sub = unary (| 0x80: one-piece exponential)
  DVM_LK_STGI,                                           // store ACC converted to i32 (sub 1) or u8 (sub 2): the same fields
  DVM_LK_STA,                                            // L[tmp] = ACC               w1 = byte offset of the temporary in a tile slot
  DVM_LK_LSS,                                            // S[a] = loaded row scalar   w1 = byte offset of its word in a tile slot (thread 0's)
  DVM_LK_STS,                                            // store S[a] per row         w1 = operand descriptor (word offset from the program)
  DVM_LK_BCS,                                            // ACC = broadcast(S[a])
  DVM_LK_SOP,                                            // per-row scalar arithmetic  sub = kind, a = dst; w1, w2, w3 as in the bytecode
  DVM_LK_PHASE,                                          // phased programs (DVM_OP_PHASE): the tiles of phases < a end here
  DVM_LK_CMP,                                            // ACC = ACC cmp Y ? 1 : 0 (Table 1, Cmp)   sub = relation, a = kind of Y (1 fp32 image,
                                                         //   2 private, 3 ACC itself), w1 = operand word                 (HEAVY variants)
  DVM_LK_SEL,                                            // Table 1, Select         sub = form (as DVM_OP_SEL + form), a = kind(p) | kind(q) << 2,
                                                         //   w1, w2 = operand words of p and q                          (HEAVY variants)
  DVM_LK_N
};

// Phased programs (rows longer than a tile): the phase tag of the bytecode travels in the top four bits of record
// word 0 (RED: bits 28..31, below them the post-operation flag; STG / STGI / STS / SOP: bits 24..27 = b).
// record word 0
#define DVM_LK_W0(h, sub, a, b) ((uint32_t)(h) | ((uint32_t)(sub) << 8) | ((uint32_t)(a) << 16) | ((uint32_t)(b) << 24))
// operand word of a local register: byte offset in the slot | mode << 18 | (fp32 ? 1 : 0) << 21 | address phase << 22 | operand << 26
#define DVM_LK_OPW(off, mode, f32, base_lo, opd) \
  ((uint32_t)(off) | ((uint32_t)(mode) << 18) | ((uint32_t)(f32) << 21) | ((uint32_t)(base_lo) << 22) | ((uint32_t)(opd) << 26))
